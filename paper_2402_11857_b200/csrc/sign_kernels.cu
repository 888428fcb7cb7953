// Scaled-sign operator (Def. 4 / Def. 5) and the server pass that consumes sign messages.
//
//   sign_uplink_kernel     p^i = C(g^i): sign words + per-tile binary64 partial of ||g||_1
//   scale_finalize_kernel  combines tile partials in tree order, scale = ||x||_1 / n
//   server_dense_kernel    v = e + (1/N) sum_i p^i for sign / identity uplinks, fused with
//                          the first half of a sign downlink (words of v, partials of ||v||_1)
//   sign_error_kernel      e <- v - p for a sign downlink
#include "device_common.cuh"
#include "kernels.h"

namespace liec {

// ------------------------------------------------------------------------------------------------
// Uplink: one CTA per (tile, worker).  Reads g once; writes 1 bit per element and one double.
// ------------------------------------------------------------------------------------------------
template <typename GT>
__global__ void __launch_bounds__(THREADS) sign_uplink_kernel(const __grid_constant__ Params p) {
    __shared__ double warp_sums[8];
    const int worker = blockIdx.y;
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int64_t row_beg = (int64_t)worker * p.d + ti.seg_beg;  // segment start in the [N][d] array
    const GT *tile_ptr = reinterpret_cast<const GT *>(p.G) + row_beg + ti.rel;
    const bool fast = (ti.len == TILE) && ((row_beg & 3) == 0);
    uint32_t *words = p.up_words + (int64_t)worker * p.W + __ldg(p.word_off + ti.t) + ti.rel / 32;
    const double s = sign_tile(tile_ptr, ti.len, fast, words, warp_sums);
    if (threadIdx.x == 0) p.up_partials[(int64_t)worker * p.TT + blockIdx.x] = s;
}

// bfloat16 gradients.  A CTA walks UPLINK_TPC consecutive tiles of one worker through a two-stage
// pipeline: each 16 KB tile is staged in shared memory by one TMA bulk copy (cp.async.bulk + an
// mbarrier per buffer), and the copy of tile i+2 is issued as soon as tile i has been consumed, so
// the table lookups and the copy latency of the next tiles hide behind the arithmetic of this one.
// Thread q owns elements 32q..32q+31 of the tile: its sign word needs no shuffles, five tree
// levels are summed in-thread and one coalesced store writes the warp's 32 words.  The four
// 16-byte chunks of a thread are read in an order XOR-rotated by the lane (bank conflicts); an XOR
// permutes the leaves of the chunk-level tree only inside its own pairs, so the sum is unchanged.
// One thread polls the mbarrier with a bounded wait; the others sleep at the CTA barrier.
constexpr int UPLINK_TPC = 4;

__global__ void __launch_bounds__(THREADS) sign_uplink_bf16_kernel(const __grid_constant__ Params p) {
    __shared__ __align__(128) unsigned short tile_s[2][TILE];
    __shared__ __align__(8) unsigned long long bar[2];
    __shared__ int64_t t_src[UPLINK_TPC], t_words[UPLINK_TPC];  // per tile: first element in the row, first word in the row's message
    __shared__ int t_len[UPLINK_TPC], t_fast[UPLINK_TPC];
    __shared__ int copy_ok;
    __shared__ double warp_sums[8];
    const int worker = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tile0 = blockIdx.x * UPLINK_TPC;
    const int ntiles = min(UPLINK_TPC, p.TT - tile0);
    const unsigned short *row = reinterpret_cast<const unsigned short *>(p.G) + (int64_t)worker * p.d;
    const bool row_aligned = (((int64_t)worker * p.d) & 7) == 0;

    // all table lookups of this CTA's tiles at once, off the per-tile critical path
    if ((int)threadIdx.x < ntiles) {
        const TileInfo tn = locate_tile(p, tile0 + threadIdx.x);
        t_src[threadIdx.x] = tn.seg_beg + tn.rel;
        t_words[threadIdx.x] = __ldg(p.word_off + tn.t) + tn.rel / 32;
        t_len[threadIdx.x] = tn.len;
        t_fast[threadIdx.x] = (tn.len == TILE && row_aligned && (tn.seg_beg & 7) == 0) ? 1 : 0;  // a 16-byte aligned full tile
    }
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[0])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[1])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        copy_ok = 1;
    }
    __syncthreads();

    uint32_t phase = 0u, pending = 0u;  // thread 0: bit b = parity of the next wait on / a copy in flight into buffer b
    // thread 0: start the copy of tile tile0 + i into buffer i & 1, if that tile takes the bulk path
    auto issue = [&](int i) {
        if (t_fast[i]) {
            pending |= 1u << (i & 1);
            const uint32_t bytes = TILE * sizeof(unsigned short);
            bulk_copy_g2s(tile_s[i & 1], row + t_src[i], bytes, bytes + p.copy_expect_extra, &bar[i & 1]);
        }
    };
    auto wait_for = [&](int buf) -> bool {  // thread 0: bounded wait for the copy in flight into buffer buf
        const bool done = mbar_wait_bounded(&bar[buf], (phase >> buf) & 1u, p.copy_wait_limit);
        if (done) { phase ^= 1u << buf; pending &= ~(1u << buf); }
        return done;
    };
    if (threadIdx.x == 0) {
        issue(0);
        if (ntiles > 1) issue(1);
    }

    for (int i = 0; i < ntiles; ++i) {
        const int buf = i & 1;
        const int len = t_len[i];
        if (t_fast[i]) {
            if (threadIdx.x == 0 && !wait_for(buf)) {
                // a copy that does not land is flagged; both buffers' copies get one more bounded
                // wait so that nothing is in flight into this CTA's shared memory when it leaves
                atomicOr(p.status, STATUS_COPY_TIMEOUT);
                if (pending & (1u << (buf ^ 1))) mbar_drain(&bar[buf ^ 1], (phase >> (buf ^ 1)) & 1u);
                mbar_drain(&bar[buf], (phase >> buf) & 1u);
                copy_ok = 0;
            }
        } else {
            const int64_t src = t_src[i];
            stage_tile_guarded(tile_s[buf], row + src, len, row_aligned && (src & 7) == 0);
        }
        __syncthreads();
        if (!copy_ok) return;

        const int pos0 = 32 * threadIdx.x;
        const int rot = (lane >> 1) & 3;
        double cs[4];
        uint32_t word = 0;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const int c = kk ^ rot;
            const uint4 q = *reinterpret_cast<const uint4 *>(&tile_s[buf][pos0 + 8 * c]);
            const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
            double d[8];
            uint32_t byte = 0;
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const float lo = __uint_as_float(w4[m] << 16), hi = __uint_as_float(w4[m] & 0xffff0000u);
                if (lo < 0.0f) byte |= 1u << (2 * m);
                if (hi < 0.0f) byte |= 2u << (2 * m);
                d[2 * m] = (double)fabsf(lo);
                d[2 * m + 1] = (double)fabsf(hi);
            }
            cs[kk] = __dadd_rn(__dadd_rn(__dadd_rn(d[0], d[1]), __dadd_rn(d[2], d[3])),
                               __dadd_rn(__dadd_rn(d[4], d[5]), __dadd_rn(d[6], d[7])));
            word |= byte << (8 * c);
        }
        // cs[kk] is chunk kk ^ rot: pairs (0,1), (2,3) stay pairs, only their order may swap
        double sum = __dadd_rn(__dadd_rn(cs[0], cs[1]), __dadd_rn(cs[2], cs[3]));
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) sum = __dadd_rn(sum, shfl_xor_f64(sum, m));

        if ((int)threadIdx.x < ((len + 31) >> 5)) p.up_words[(int64_t)worker * p.W + t_words[i] + threadIdx.x] = word;
        if (lane == 0) warp_sums[warp] = sum;
        __syncthreads();  // the buffer has been read by everyone; the warp sums are in place
        if (threadIdx.x == 0 && i + 2 < ntiles) issue(i + 2);
        if (threadIdx.x == 32) {  // (not thread 0: it is busy with the copies)
            const double s01 = __dadd_rn(warp_sums[0], warp_sums[1]), s23 = __dadd_rn(warp_sums[2], warp_sums[3]);
            const double s45 = __dadd_rn(warp_sums[4], warp_sums[5]), s67 = __dadd_rn(warp_sums[6], warp_sums[7]);
            p.up_partials[(int64_t)worker * p.TT + tile0 + i] = __dadd_rn(__dadd_rn(s01, s23), __dadd_rn(s45, s67));
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Scale: one CTA per (segment, row).  Tile partials are combined in tree order
// (tree_reduce_partials), then scale = S / n.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS) scale_finalize_kernel(const __grid_constant__ Params p,
                                                                  const double *partials, float *scales,
                                                                  double *sums /* when set: the plain sums instead */) {
    __shared__ double buf[FIN_CHUNK];
    __shared__ double chunk_sums[FIN_MAX_CHUNKS];
    const int t = blockIdx.x, row = blockIdx.y;
    const int first = __ldg(p.tile_prefix + t);
    const int ntiles = __ldg(p.tile_prefix + t + 1) - first;
    const double total = tree_reduce_partials(partials + (int64_t)row * p.TT + first, ntiles, buf, chunk_sums);
    if (threadIdx.x == 0) {
        const int64_t n = __ldg(p.seg_off + t + 1) - __ldg(p.seg_off + t);
        if (sums) {
            sums[(int64_t)row * p.T + t] = total;
        } else {
            scales[(int64_t)row * p.T + t] = __double2float_rn(__ddiv_rn(total, (double)n));
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Server pass for an identity uplink (the messages are the raw gradients): one CTA per tile.
//   acc = +0; for i = 0..N-1: acc = acc + p^i_j;   v_j = e_j + acc / N        (written over e)
// and, when the downlink is scaled sign, the words of v and the tile partial of ||v||_1.
// ------------------------------------------------------------------------------------------------
// TEL: also the tile's partial sums of e^2 (as read) and v^2 (as written), same tree as the L1 norm.
template <bool DOWN_SIGN, typename GT, bool TEL>
__global__ void __launch_bounds__(THREADS) server_dense_kernel(const __grid_constant__ Params p) {
    __shared__ double warp_sums[8];
    __shared__ double tel_sums[TEL ? 16 : 1];
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0);
    const int64_t wbase = __ldg(p.word_off + ti.t) + ti.rel / 32;
    const int nwords = (ti.len + 31) >> 5;

    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[j][c] = 0.0f;

    {  // identity uplink: the message is the gradient itself
        // (one answer for all workers, so that the loop carries no branch and its loads pipeline)
        const bool gfast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0) && ((p.d & 3) == 0);
#pragma unroll 2
        for (int i = 0; i < p.N; ++i) {
            const int64_t row_beg = (int64_t)i * p.d + ti.seg_beg;
            const GT *tile_ptr = reinterpret_cast<const GT *>(p.G) + row_beg + ti.rel;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float g[4];
                if (gfast) load4_stream(tile_ptr + tile_pos(warp, lane, j), g);
                else load4_guarded(tile_ptr, tile_pos(warp, lane, j), ti.len, g);
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[j][c] = __fadd_rn(acc[j][c], g[c]);
            }
        }
    }

    const WorkerDivisor by_n(p.N);
    float *e_tile = p.e + ti.seg_beg + ti.rel;
    double a[8];
    double te[TEL ? 8 : 1], tv[TEL ? 8 : 1];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
        float ev[4], v[4];
        if (fast) load4_stream(e_tile + pos, ev);
        else load4_guarded(e_tile, pos, ti.len, ev);
        if constexpr (TEL) te[j] = leaf4_sq(ev);
        by_n.div4(acc[j], v);
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = __fadd_rn(ev[c], v[c]);
        if (fast) {
            *reinterpret_cast<float4 *>(e_tile + pos) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (pos + c < ti.len) e_tile[pos + c] = v[c]; else v[c] = 0.0f;  // padding: +0, bit 0
            }
        }
        if constexpr (TEL) tv[j] = leaf4_sq(v);
        if (DOWN_SIGN) {
            a[j] = leaf4(v);
            uint32_t w = pack_word(sign_nibble(v), lane);
            int widx = warp * 32 + j * 4 + (lane >> 3);
            if ((lane & 7) == 0 && widx < nwords) p.down_words[wbase + widx] = w;
        }
    }
    if (DOWN_SIGN) {
        double s = cta_tree_reduce(warp_tree_reduce8(a, lane), warp_sums);
        if (threadIdx.x == 0) p.down_partials[blockIdx.x] = s;
    }
    if constexpr (TEL) {
        double re, rv;
        cta_tree_reduce_pair(warp_tree_reduce8(te, lane), warp_tree_reduce8(tv, lane), tel_sums, re, rv);
        if (threadIdx.x == 0) { p.tel_e[blockIdx.x] = re; p.tel_v[blockIdx.x] = rv; }
    }
}

// Sign uplink, one thread per 32-bit word: thread q of the CTA owns elements 32q..32q+31 of the
// tile, i.e. exactly one word of every worker's message, so unpacking needs no shuffles
// (shift + sign-xor + add per element and worker), the word of v is built in-thread and the
// ||v||_1 leaf covers five tree levels in-thread.
// Nibble k of the result is nibble k ^ m of w (m in 0..7; its own inverse).  sel = 0x3210 ^ ((m >> 1) * 0x1111).
__device__ __forceinline__ uint32_t nibble_xor_perm(uint32_t w, uint32_t m, uint32_t sel) {
    const uint32_t sw = ((w & 0x0f0f0f0fu) << 4) | ((w >> 4) & 0x0f0f0f0fu);
    return __byte_perm((m & 1u) ? sw : w, 0u, sel);
}

template <bool DOWN_SIGN, bool TEL>
__global__ void __launch_bounds__(THREADS) server_sign_kernel(const __grid_constant__ Params p) {
    __shared__ __align__(128) float tile_s[TILE];  // the tile of e, then of v
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int copy_ok;
    __shared__ double warp_sums[8];
    __shared__ double tel_sums[TEL ? 16 : 1];
    constexpr int SCALE_CHUNK = 1024;              // workers whose scales are staged at once (a multiple of WG)
    __shared__ float up_scale_smem[SCALE_CHUNK];   // this segment's scales of workers c0 .. c0 + SCALE_CHUNK - 1
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0);
    const int64_t wbase = __ldg(p.word_off + ti.t) + ti.rel / 32;
    const int nwords = (ti.len + 31) >> 5;
    const int my_widx = threadIdx.x;
    const bool have_word = my_widx < nwords;
    float *e_tile = p.e + ti.seg_beg + ti.rel;

    // Thread q owns word q of the tile = elements 32q .. 32q+31, which it reads from shared memory as
    // eight 16-byte chunks; the tile comes in by one bulk copy (or guarded loads for a ragged or
    // misaligned tile) and v leaves by coalesced stores, so no global access is strided.  To keep the
    // shared-memory reads free of bank conflicts the thread takes its chunks in the order k ^ (q & 7),
    // and permutes the nibbles of every sign word the same way: slot (k, j) of its registers is then
    // element 4 (k ^ (q & 7)) + j throughout.  The binary64 tree over a thread's eight chunks does not
    // see the order: a XOR permutation of the leaves only swaps the operands of additions.
    const uint32_t rot = threadIdx.x & 7u;
    const uint32_t rot_sel = 0x3210u ^ ((rot >> 1) * 0x1111u);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        copy_ok = 1;
        if (fast) {
            const uint32_t bytes = TILE * sizeof(float);
            bulk_copy_g2s(tile_s, e_tile, bytes, bytes + p.copy_expect_extra, &bar);
        }
    }
    if (!fast) stage_tile_guarded(tile_s, e_tile, ti.len, (ti.seg_beg & 3) == 0);

    // The first 8 workers' contribution to an element depends only on their 8 sign bits there: the
    // running sum ((+0 + p^0) + p^1) + ... + p^7 is tabulated once per CTA for the 256 bit patterns (entry
    // t by thread t, the same additions in the same order), and an element looks its pattern up.  The
    // patterns of a thread's 32 elements come from a bit transposition of its 8 words: X[c] holds, in
    // byte k, the pattern of slot c + 8k.  The workers after the eighth are added one by one.
    constexpr int HEAD = 8;
    __shared__ float head_sum[1 << HEAD];
    static_assert(THREADS == (1 << HEAD), "one table entry per thread");
    const uint32_t *wp = p.up_words + wbase + my_widx;
    uint32_t hw[HEAD];
#pragma unroll
    for (int r = 0; r < HEAD; ++r) hw[r] = (have_word && r < p.N) ? __ldg(wp + (int64_t)r * p.W) : 0u;
    // workers four at a time: their four words are fetched together, one group ahead of use
    constexpr int WG = 4;
    uint32_t nextw[WG];
#pragma unroll
    for (int u = 0; u < WG; ++u) nextw[u] = (have_word && HEAD + u < p.N) ? __ldg(wp + (int64_t)(HEAD + u) * p.W) : 0u;
    for (int i = threadIdx.x; i < SCALE_CHUNK && i < p.N; i += THREADS) up_scale_smem[i] = p.up_scales[(int64_t)i * p.T + ti.t];
    __syncthreads();
    {
        float a = 0.0f;
#pragma unroll
        for (int r = 0; r < HEAD; ++r)
            if (r < p.N) a = __fadd_rn(a, __uint_as_float(__float_as_uint(up_scale_smem[r]) ^ (((threadIdx.x >> r) & 1u) << 31)));
        head_sum[threadIdx.x] = a;   // (bits of absent workers are zero in every pattern)
    }
    __syncthreads();
    float acc[32];
    {
        uint32_t X[8];
#pragma unroll
        for (int r = 0; r < HEAD; ++r) hw[r] = nibble_xor_perm(hw[r], rot, rot_sel);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            X[c] = 0u;
#pragma unroll
            for (int r = 0; r < HEAD; ++r) X[c] |= (r >= c ? hw[r] << (r - c) : hw[r] >> (c - r)) & (0x01010101u << r);
        }
#pragma unroll
        for (int c = 0; c < 32; ++c) acc[c] = head_sum[(X[c & 7] >> (8 * (c >> 3))) & 0xffu];
    }
    for (int i0 = HEAD; i0 < p.N; i0 += WG) {
        if ((i0 & (SCALE_CHUNK - 1)) == 0) {  // (uniform over the CTA) next chunk of scales
            __syncthreads();
            for (int i = threadIdx.x; i < SCALE_CHUNK && i0 + i < p.N; i += THREADS)
                up_scale_smem[i] = p.up_scales[(int64_t)(i0 + i) * p.T + ti.t];
            __syncthreads();
        }
        uint32_t w[WG];
#pragma unroll
        for (int u = 0; u < WG; ++u) w[u] = nibble_xor_perm(nextw[u], rot, rot_sel);
#pragma unroll
        for (int u = 0; u < WG; ++u) {
            const int i = i0 + WG + u;
            nextw[u] = (have_word && i < p.N) ? __ldg(wp + (int64_t)i * p.W) : 0u;
        }
#pragma unroll
        for (int u = 0; u < WG; ++u) {
            if (i0 + u < p.N) {  // uniform over the CTA
                const uint32_t sbits = __float_as_uint(up_scale_smem[(i0 + u) & (SCALE_CHUNK - 1)]);
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float pij = __uint_as_float(sbits ^ ((w[u] << (31 - c)) & 0x80000000u));
                    acc[c] = __fadd_rn(acc[c], pij);
                }
            }
        }
    }

    // the tile of e must have landed by now
    if (fast && threadIdx.x == 0 && !mbar_wait_bounded(&bar, 0u, p.copy_wait_limit)) {
        atomicOr(p.status, STATUS_COPY_TIMEOUT);
        mbar_drain(&bar, 0u);
        copy_ok = 0;
    }
    __syncthreads();
    if (!copy_ok) return;   // (nothing has been written)

    const WorkerDivisor by_n(p.N);
    const int pos0 = 32 * threadIdx.x;
    uint32_t vword = 0u;
    double leaf[8];
    double te[TEL ? 8 : 1], tv[TEL ? 8 : 1];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int pos = pos0 + 4 * (k ^ (int)rot);
        float ev[4], v[4];
        {
            const float4 q = *reinterpret_cast<const float4 *>(&tile_s[pos]);
            ev[0] = q.x; ev[1] = q.y; ev[2] = q.z; ev[3] = q.w;
        }
        if constexpr (TEL) te[k] = leaf4_sq(ev);
        {
            const float a4[4] = {acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]};
            by_n.div4(a4, v);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            v[c] = __fadd_rn(ev[c], v[c]);
            if (!fast && pos + c >= ti.len) v[c] = 0.0f;
        }
        *reinterpret_cast<float4 *>(&tile_s[pos]) = make_float4(v[0], v[1], v[2], v[3]);
        if constexpr (TEL) tv[k] = leaf4_sq(v);
        if (DOWN_SIGN) {
            leaf[k] = leaf4(v);
            vword |= sign_nibble(v) << (4 * k);
        }
    }
    __syncthreads();
    // v over e, coalesced
    if (fast) {
#pragma unroll
        for (int c = 0; c < TILE / 4 / THREADS; ++c) {
            const int q = c * THREADS + threadIdx.x;
            reinterpret_cast<float4 *>(e_tile)[q] = reinterpret_cast<const float4 *>(tile_s)[q];
        }
    } else {
        for (int q = threadIdx.x; q < ti.len; q += THREADS) e_tile[q] = tile_s[q];
    }
    // a thread's 32 consecutive elements: three more tree levels in-thread, five across the lanes
    auto thread_then_warp = [](const double (&l)[8]) {
        double s = __dadd_rn(__dadd_rn(__dadd_rn(l[0], l[1]), __dadd_rn(l[2], l[3])),
                             __dadd_rn(__dadd_rn(l[4], l[5]), __dadd_rn(l[6], l[7])));
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) s = __dadd_rn(s, shfl_xor_f64(s, m));
        return s;
    };
    if (DOWN_SIGN) {
        if (have_word) p.down_words[wbase + my_widx] = nibble_xor_perm(vword, rot, rot_sel);
        const double s = cta_tree_reduce(thread_then_warp(leaf), warp_sums);
        if (threadIdx.x == 0) p.down_partials[blockIdx.x] = s;
    }
    if constexpr (TEL) {
        double re, rv;
        cta_tree_reduce_pair(thread_then_warp(te), thread_then_warp(tv), tel_sums, re, rv);
        if (threadIdx.x == 0) { p.tel_e[blockIdx.x] = re; p.tel_v[blockIdx.x] = rv; }
    }
}

// ------------------------------------------------------------------------------------------------
// Global error for a sign downlink: e_j <- v_j - p_j with p_j = -s or +s by the sign word.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS) sign_error_kernel(const __grid_constant__ Params p) {
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0);
    const int64_t wbase = __ldg(p.word_off + ti.t) + ti.rel / 32;
    const int nwords = (ti.len + 31) >> 5;
    const float s = p.down_scales[ti.t];
    const uint32_t sbits = __float_as_uint(s);
    float *e_tile = p.e + ti.seg_beg + ti.rel;
    const int my_widx = warp * 32 + lane;
    const uint32_t my_word = my_widx < nwords ? p.down_words[wbase + my_widx] : 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
        uint32_t nib = nibble_from_words(my_word, lane, j);
        float v[4];
        if (fast) load4_stream(e_tile + pos, v);
        else load4_guarded(e_tile, pos, ti.len, v);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float pj = __uint_as_float(sbits ^ ((nib << (31 - c)) & 0x80000000u));
            v[c] = __fsub_rn(v[c], pj);
        }
        if (fast) {
            *reinterpret_cast<float4 *>(e_tile + pos) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (pos + c < ti.len) e_tile[pos + c] = v[c];
        }
    }
}

// Identity downlink: p = v, so the workers read v from a copy and the error becomes +0.
__global__ void __launch_bounds__(THREADS) identity_downlink_kernel(const __grid_constant__ Params p) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < p.d; j += stride) {
        p.vbuf[j] = p.e[j];
        p.e[j] = 0.0f;
    }
}

// ------------------------------------------------------------------------------------------------
// Squared norms per tile (monitoring): leaves x^2 in binary64 (exact), same tree as the L1 norm.
// ------------------------------------------------------------------------------------------------
template <typename GT>
__global__ void __launch_bounds__(THREADS) sumsq_kernel(const __grid_constant__ Params p, const GT *src,
                                                         const int64_t row_stride) {
    __shared__ double warp_sums[8];
    const int row = blockIdx.y;
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row_beg = (int64_t)row * row_stride + ti.seg_beg;
    const GT *tile_ptr = src + row_beg + ti.rel;
    // (the source may be a message buffer, whose rows start on 4-byte boundaries only: look at the address)
    const bool fast = (ti.len == TILE) && ((reinterpret_cast<uintptr_t>(tile_ptr) & (4 * sizeof(GT) - 1)) == 0);
    double a[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float v[4];
        if (fast) load4_stream(tile_ptr + tile_pos(warp, lane, j), v);
        else load4_guarded(tile_ptr, tile_pos(warp, lane, j), ti.len, v);
        a[j] = leaf4_sq(v);
    }
    double s = cta_tree_reduce(warp_tree_reduce8(a, lane), warp_sums);
    if (threadIdx.x == 0) p.tel_partials[(int64_t)row * p.TT + blockIdx.x] = s;
}

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
cudaError_t launch_sumsq(const Params &p, const void *src, int64_t row_stride, int rows, bool bf16, cudaStream_t st) {
    dim3 grid(p.TT, rows);
    if (bf16) sumsq_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(p, static_cast<const __nv_bfloat16 *>(src), row_stride);
    else sumsq_kernel<float><<<grid, THREADS, 0, st>>>(p, static_cast<const float *>(src), row_stride);
    return cudaGetLastError();
}

cudaError_t launch_sum_finalize(const Params &p, const double *partials, int rows, double *out, cudaStream_t st) {
    dim3 grid(p.T, rows);
    scale_finalize_kernel<<<grid, THREADS, 0, st>>>(p, partials, nullptr, out);
    return cudaGetLastError();
}

cudaError_t launch_sign_uplink(const Params &p, cudaStream_t st) {
    dim3 grid(p.TT, p.N);
    if (p.gdt == DT_F32) sign_uplink_kernel<float><<<grid, THREADS, 0, st>>>(p);
    else sign_uplink_bf16_kernel<<<dim3((p.TT + UPLINK_TPC - 1) / UPLINK_TPC, p.N), THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_scale_finalize(const Params &p, bool uplink, cudaStream_t st) {
    dim3 grid(p.T, uplink ? p.N : 1);
    scale_finalize_kernel<<<grid, THREADS, 0, st>>>(p, uplink ? p.up_partials : p.down_partials,
                                                    uplink ? p.up_scales : p.down_scales, nullptr);
    return cudaGetLastError();
}

template <typename GT, bool TEL>
static cudaError_t launch_server_dense_t(const Params &p, cudaStream_t st) {
    if (p.down == COMP_SIGN) server_dense_kernel<true, GT, TEL><<<p.TT, THREADS, 0, st>>>(p);
    else server_dense_kernel<false, GT, TEL><<<p.TT, THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

template <bool TEL>
static cudaError_t launch_server_dense_tel(const Params &p, cudaStream_t st) {
    if (p.up == COMP_SIGN) {
        if (p.down == COMP_SIGN) server_sign_kernel<true, TEL><<<p.TT, THREADS, 0, st>>>(p);
        else server_sign_kernel<false, TEL><<<p.TT, THREADS, 0, st>>>(p);
        return cudaGetLastError();
    }
    if (p.gdt == DT_F32) return launch_server_dense_t<float, TEL>(p, st);
    return launch_server_dense_t<__nv_bfloat16, TEL>(p, st);
}

cudaError_t launch_server_dense(const Params &p, cudaStream_t st) {
    return p.telemetry ? launch_server_dense_tel<true>(p, st) : launch_server_dense_tel<false>(p, st);
}

cudaError_t launch_sign_error(const Params &p, cudaStream_t st) {
    sign_error_kernel<<<p.TT, THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_identity_downlink(const Params &p, cudaStream_t st) {
    int64_t blocks = (p.d + THREADS - 1) / THREADS;
    if (blocks > 148 * 16) blocks = 148 * 16;
    identity_downlink_kernel<<<(int)blocks, THREADS, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace liec
