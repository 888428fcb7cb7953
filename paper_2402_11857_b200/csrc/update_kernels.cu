// Local immediate error compensation and model update (last worker step of Algorithm 1):
//   x^i_j <- x^i_j - eta * ((p_j - p^i_j) + g^i_j)
// p^i is not stored: it is recomputed from g^i and the worker's own scale (sign), its
// selection threshold (top-k), its subset (random-k, decoded from the index list into a bit mask
// of the tile) or taken as g^i itself (identity).  p is decoded from the downlink message; a
// random-k downlink has the top-k layout and takes the top-k path (DOWN == COMP_TOPK).
#include "device_common.cuh"
#include "kernels.h"

namespace liec {

// TEL: the kernel also leaves, per (worker, tile), the binary64 partial sum of g^2 over the tile's
// part of the summation tree (the gradient is in registers here anyway).
template <int UP, int DOWN, typename GT, bool TEL>
__global__ void __launch_bounds__(THREADS, (DOWN == COMP_TOPK || TEL ? 3 : 0)) worker_update_kernel(const __grid_constant__ Params p, const float lr) {
    __shared__ __align__(16) float p_tile[DOWN == COMP_TOPK ? TILE : 4];  // decoded downlink message (top-k)
    // With a top-k downlink a CTA serves WPC workers so that the message is decoded once for them.
    constexpr int WPC = DOWN == COMP_TOPK ? 4 : 1;
    __shared__ double tel_sums[TEL ? WPC : 1][TEL ? 8 : 1];
    __shared__ uint32_t own_mask[UP == COMP_RANDK ? WPC : 1][UP == COMP_RANDK ? TILE_WORDS : 1];  // each worker's own subset inside this tile
    // (a sparse downlink: the tile's range in the message is fetched first, so that the entries themselves can be
    // requested right behind the first worker's streaming loads instead of two latencies later)
    uint32_t down_beg = 0, down_end_next = 0;
    if (DOWN == COMP_TOPK) {
        down_beg = p.down_outbase[blockIdx.x];
        down_end_next = p.down_outbase[blockIdx.x + 1];   // ([TT + 1] entries; the segment's last tile ends at its k-range instead)
    }
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int wq = 0; wq < WPC; ++wq) {
    const int worker = blockIdx.y * WPC + wq;
    if (worker >= p.N) break;
    const int64_t row_beg = (int64_t)worker * p.d + ti.seg_beg;
    const bool fast = (ti.len == TILE) && ((row_beg & 3) == 0);
    const GT *g_tile = reinterpret_cast<const GT *>(p.G) + row_beg + ti.rel;
    float *x_tile = p.X + row_beg + ti.rel;

    float su = 0.0f, sd = 0.0f;
    uint32_t my_word = 0u;
    if (UP == COMP_SIGN) su = p.up_scales[(int64_t)worker * p.T + ti.t];
    if (DOWN == COMP_SIGN) {
        sd = p.down_scales[ti.t];
        const int nwords = (ti.len + 31) >> 5;
        const int my_widx = warp * 32 + lane;
        if (my_widx < nwords) my_word = __ldg(p.down_words + __ldg(p.word_off + ti.t) + ti.rel / 32 + my_widx);
    }
    const uint32_t su_bits = __float_as_uint(su), sd_bits = __float_as_uint(sd);
    uint32_t up_thresh = 0u, up_cut = 0u;
    if (UP == COMP_TOPK) {  // the worker's own selection rule: |g| above the threshold, ties up to the cut index
        const uint32_t *sel = p.up_sel + ((int64_t)worker * p.T + ti.t) * SEL_WORDS;
        up_thresh = sel[SEL_THRESH];
        up_cut = sel[SEL_CUT];
    }
    // element c of a quad whose first flat index is r is kept iff key > T, or key == T and r + c <= cut, i.e.
    // ~r >= ~cut + c (which cannot wrap when cut >= c; when cut < c no index r + c can be at or below the cut and
    // the bound asks for key > T alone)
    unsigned long long kept_bound[4];
#pragma unroll
    for (int c = 0; c < 4; ++c)
        kept_bound[c] = up_cut >= (uint32_t)c ? (((unsigned long long)up_thresh << 32) | (uint32_t)(~up_cut + (uint32_t)c))
                                               : ((unsigned long long)(up_thresh + 1u) << 32);
    const float *v_tile = DOWN == COMP_IDENTITY ? p.vbuf + ti.seg_beg + ti.rel : nullptr;

    float g[8][4], x[8][4];
    if (fast) {
#pragma unroll
        for (int j = 0; j < 8; ++j) load4_stream(g_tile + tile_pos(warp, lane, j), g[j]);
#pragma unroll
        for (int j = 0; j < 8; ++j) load4_stream(x_tile + tile_pos(warp, lane, j), x[j]);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            load4_guarded(g_tile, tile_pos(warp, lane, j), ti.len, g[j]);
            load4_guarded(x_tile, tile_pos(warp, lane, j), ti.len, x[j]);
        }
    }

    // decode the downlink top-k message of this tile (after the streaming loads are in flight)
    if (DOWN == COMP_TOPK && wq == 0) {
        const bool last_tile = (blockIdx.x + 1 == __ldg(p.tile_prefix + ti.t + 1));
        const uint32_t beg = down_beg;
        const uint32_t end = last_tile ? (uint32_t)__ldg(p.k_off + ti.t + 1) : down_end_next;
        const uint32_t tile_first = (uint32_t)(ti.seg_beg + ti.rel);
        // the first entry of every thread is requested before the tile is cleared
        const uint32_t q0 = beg + threadIdx.x;
        uint32_t o0 = 0xffffffffu;
        float val0 = 0.0f;
        if (q0 < end) { o0 = p.down_idx[q0] - tile_first; val0 = p.down_val[q0]; }
        for (int q = threadIdx.x; q < TILE / 4; q += THREADS)
            reinterpret_cast<float4 *>(p_tile)[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        __syncthreads();
        if (o0 < (uint32_t)TILE) p_tile[o0] = val0;
        for (uint32_t q = q0 + THREADS; q < end; q += THREADS) {
            const uint32_t o = p.down_idx[q] - tile_first;
            if (o < (uint32_t)TILE) p_tile[o] = p.down_val[q];
        }
        __syncthreads();
    }
    if (UP == COMP_RANDK && wq == 0) {  // the subsets of all of this CTA's workers, decoded together
#pragma unroll
        for (int u = 0; u < WPC; ++u) own_mask[u][threadIdx.x] = 0u;   // THREADS == TILE_WORDS
        __syncthreads();
        const bool last_tile = (blockIdx.x + 1 == __ldg(p.tile_prefix + ti.t + 1));
        const uint32_t tile_first = (uint32_t)(ti.seg_beg + ti.rel);
#pragma unroll
        for (int u = 0; u < WPC; ++u) {
            const int wu = blockIdx.y * WPC + u;
            if (wu < p.N) {
                const uint32_t *ob = p.up_outbase + (int64_t)wu * (p.TT + 1) + blockIdx.x;
                const uint32_t beg = ob[0];
                const uint32_t end = last_tile ? (uint32_t)__ldg(p.k_off + ti.t + 1) : ob[1];
                const uint32_t *own_idx = p.up_idx + (int64_t)wu * p.K;
                for (uint32_t q = beg + threadIdx.x; q < end; q += THREADS) {
                    const uint32_t o = own_idx[q] - tile_first;
                    if (o < (uint32_t)TILE) atomicOr(&own_mask[u][o >> 5], 1u << (o & 31));
                }
            }
        }
        __syncthreads();
    }

    double tg[TEL ? 8 : 1];   // TEL: this lane's sums of g^2, row by row, as the rows are consumed
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
        if constexpr (TEL) tg[j] = leaf4_sq(g[j]);
        float pd[4];
        if (DOWN == COMP_SIGN) {
            uint32_t nib = nibble_from_words(my_word, lane, j);
#pragma unroll
            for (int c = 0; c < 4; ++c) pd[c] = __uint_as_float(sd_bits ^ ((nib << (31 - c)) & 0x80000000u));
        } else if (DOWN == COMP_IDENTITY) {
            load4_guarded(v_tile, pos, ti.len, pd);
        } else {
            const float4 q4 = *reinterpret_cast<const float4 *>(&p_tile[pos]);
            pd[0] = q4.x; pd[1] = q4.y; pd[2] = q4.z; pd[3] = q4.w;
        }
        uint32_t own_nib = 0u;
        if (UP == COMP_RANDK) own_nib = own_mask[wq][pos >> 5] >> (pos & 31);  // pos is a multiple of 4: the four bits share a word
        // top-k: kept <=> (key, ~index) >= (threshold, ~cut) as one 64-bit comparison; the row's index part is
        // formed once, the per-element offset sits in the bound (see kept_bound)
        const uint32_t row_low = ~((uint32_t)(ti.seg_beg + ti.rel) + (uint32_t)pos);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float pi;
            if (UP == COMP_RANDK) {
                pi = ((own_nib >> c) & 1u) ? g[j][c] : 0.0f;
            } else if (UP == COMP_SIGN) {
                pi = __uint_as_float(su_bits ^ (g[j][c] < 0.0f ? 0x80000000u : 0u));
            } else if (UP == COMP_TOPK) {
                const uint32_t key = __float_as_uint(g[j][c]) & 0x7fffffffu;
                const bool kept = (((unsigned long long)key << 32) | row_low) >= kept_bound[c];
                pi = kept ? g[j][c] : 0.0f;
            } else {
                pi = g[j][c];
            }
            float diff = __fsub_rn(pd[c], pi);
            float u = __fadd_rn(diff, g[j][c]);
            x[j][c] = __fsub_rn(x[j][c], __fmul_rn(lr, u));
        }
        if (fast) {
            __stcs(reinterpret_cast<float4 *>(x_tile + pos), make_float4(x[j][0], x[j][1], x[j][2], x[j][3]));
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (pos + c < ti.len) x_tile[pos + c] = x[j][c];
        }
    }
    if constexpr (TEL) {
        const double s = cta_tree_reduce(warp_tree_reduce8(tg, lane), tel_sums[wq]);
        if (threadIdx.x == 0) p.tel_g[(int64_t)worker * p.TT + blockIdx.x] = s;
    }
    }  // workers of this CTA
}

template <int UP, int DOWN>
static cudaError_t launch_t(const Params &p, float lr, cudaStream_t st) {
    constexpr int WPC = DOWN == COMP_TOPK ? 4 : 1;
    dim3 grid(p.TT, (p.N + WPC - 1) / WPC);
    if (p.telemetry) {
        if (p.gdt == DT_F32) worker_update_kernel<UP, DOWN, float, true><<<grid, THREADS, 0, st>>>(p, lr);
        else worker_update_kernel<UP, DOWN, __nv_bfloat16, true><<<grid, THREADS, 0, st>>>(p, lr);
    } else {
        if (p.gdt == DT_F32) worker_update_kernel<UP, DOWN, float, false><<<grid, THREADS, 0, st>>>(p, lr);
        else worker_update_kernel<UP, DOWN, __nv_bfloat16, false><<<grid, THREADS, 0, st>>>(p, lr);
    }
    return cudaGetLastError();
}

cudaError_t launch_worker_update(const Params &p_in, float lr, cudaStream_t st) {
    Params p = p_in;
    if (p.down == COMP_RANDK) p.down = COMP_TOPK;  // same message layout, same decode
    if (p.up == COMP_RANDK && p.down == COMP_TOPK) return launch_t<COMP_RANDK, COMP_TOPK>(p, lr, st);
    if (p.up == COMP_RANDK && p.down == COMP_SIGN) return launch_t<COMP_RANDK, COMP_SIGN>(p, lr, st);
    if (p.up == COMP_RANDK && p.down == COMP_IDENTITY) return launch_t<COMP_RANDK, COMP_IDENTITY>(p, lr, st);
    if (p.up == COMP_SIGN && p.down == COMP_SIGN) return launch_t<COMP_SIGN, COMP_SIGN>(p, lr, st);
    if (p.up == COMP_SIGN && p.down == COMP_IDENTITY) return launch_t<COMP_SIGN, COMP_IDENTITY>(p, lr, st);
    if (p.up == COMP_IDENTITY && p.down == COMP_SIGN) return launch_t<COMP_IDENTITY, COMP_SIGN>(p, lr, st);
    if (p.up == COMP_IDENTITY && p.down == COMP_IDENTITY) return launch_t<COMP_IDENTITY, COMP_IDENTITY>(p, lr, st);
    if (p.up == COMP_TOPK && p.down == COMP_TOPK) return launch_t<COMP_TOPK, COMP_TOPK>(p, lr, st);
    if (p.up == COMP_TOPK && p.down == COMP_SIGN) return launch_t<COMP_TOPK, COMP_SIGN>(p, lr, st);
    if (p.up == COMP_TOPK && p.down == COMP_IDENTITY) return launch_t<COMP_TOPK, COMP_IDENTITY>(p, lr, st);
    if (p.up == COMP_SIGN && p.down == COMP_TOPK) return launch_t<COMP_SIGN, COMP_TOPK>(p, lr, st);
    if (p.up == COMP_IDENTITY && p.down == COMP_TOPK) return launch_t<COMP_IDENTITY, COMP_TOPK>(p, lr, st);
    return cudaErrorInvalidValue;
}

}  // namespace liec
