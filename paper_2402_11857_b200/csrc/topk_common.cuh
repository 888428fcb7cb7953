// Shared by the top-k kernels (Def. 2): the description of one side of the iteration, the status
// bits, and the block-wide helpers (histogram flush, rank pick, prefix sum).
#pragma once
#include <type_traits>

#include "device_common.cuh"
#include "philox.cuh"

namespace liec {

// Element type tag of a selection whose values are not in memory: the pseudo-random scores of the
// seeded random-k draw, computed where they are needed (as binary32 bit patterns, see philox.cuh).
struct ScoreGen { float unused; };

struct TopkSide {
    const void *src;      // rows of the vector being compressed (unused for generated scores)
    ScoreStream gen;      // generated scores: key and draw number
    int64_t row_stride;   // elements between rows (d for the uplink, 0 for the single downlink row)
    int R;                // rows
    uint32_t *idx; float *val;            // [R][K] output message
    uint32_t *hist, *hist2, *sel;         // [R][T][...]
    uint32_t *cand_idx; float *cand_val;  // [R][CAP]
    const int64_t *cap_off;                // [T+1] candidate capacity prefix of this side
    int64_t CAP, cap_long_max;             // its total; the largest capacity among the long segments
    uint32_t *meta;                        // [R][TT][4]: pos, cnt, n_greater -> unused, ties allowed
    uint32_t *outbase;                     // [R][TT+1]
    uint32_t *scan_parts;                  // [R][T][scan_parts][2]
    float *zero_out;                       // downlink: error buffer, selected entries become +0
    int spec;                              // uplink: try last step's threshold first (single dense pass)
};

inline TopkSide make_side(const Params &p, bool uplink) {
    TopkSide s;
    s.gen = ScoreStream{0u, 0u, 0u};
    if (uplink) {
        s.src = p.G; s.row_stride = p.d; s.R = p.N;
        s.idx = p.up_idx; s.val = p.up_val; s.hist = p.up_hist; s.hist2 = p.up_hist2; s.sel = p.up_sel;
        s.cand_idx = p.up_cand_idx; s.cand_val = p.up_cand_val; s.meta = p.up_tile_meta; s.outbase = p.up_outbase; s.scan_parts = p.up_scan_parts;
        s.cap_off = p.cap_off; s.CAP = p.CAP; s.cap_long_max = p.cap_long_max;
        s.zero_out = nullptr;
        s.spec = 1;
    } else {
        s.src = p.e; s.row_stride = 0; s.R = 1;
        s.idx = p.down_idx; s.val = p.down_val; s.hist = p.down_hist; s.hist2 = p.down_hist2; s.sel = p.down_sel;
        s.cand_idx = p.down_cand_idx; s.cand_val = p.down_cand_val; s.meta = p.down_tile_meta; s.outbase = p.down_outbase; s.scan_parts = p.down_scan_parts;
        s.cap_off = p.down_cap_off; s.CAP = p.down_CAP; s.cap_long_max = p.down_cap_long_max;
        s.zero_out = p.e;
        s.spec = 0;
    }
    return s;
}

__device__ __forceinline__ uint32_t key_of(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// ---- where a selection's values come from -----------------------------------------------------
// Four consecutive values of a tile at position `pos` (a multiple of 4) in the 4-wide layout;
// positions at or beyond the tile's length read as +0.
template <typename GT>
__device__ __forceinline__ void fetch4(const TopkSide &s, int row, const TileInfo &ti, int pos, float (&v)[4]) {
    if constexpr (std::is_same<GT, ScoreGen>::value) {
        const uint4 w = s.gen.block((uint32_t)((ti.rel + pos) >> 2), (uint32_t)ti.t, (uint32_t)row);
        const uint32_t w4[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = pos + c < ti.len ? __uint_as_float(w4[c]) : 0.0f;
    } else {
        const int64_t row_beg = (int64_t)row * s.row_stride + ti.seg_beg;
        const GT *tile_ptr = reinterpret_cast<const GT *>(s.src) + row_beg + ti.rel;
        if ((ti.len == TILE) && ((row_beg & 3) == 0)) load4_stream(tile_ptr + pos, v);
        else load4_guarded(tile_ptr, pos, ti.len, v);
    }
}

// One value of segment t (position j relative to the segment); the dense one-CTA path only.
template <typename GT>
__device__ __forceinline__ float fetch1(const TopkSide &s, int row, int t, int64_t seg_beg, int64_t j) {
    if constexpr (std::is_same<GT, ScoreGen>::value) {
        const uint4 w = s.gen.block((uint32_t)(j >> 2), (uint32_t)t, (uint32_t)row);
        const uint32_t w4[4] = {w.x, w.y, w.z, w.w};
        return __uint_as_float(w4[j & 3]);
    } else {
        return load1(reinterpret_cast<const GT *>(s.src) + (int64_t)row * s.row_stride + seg_beg + j);
    }
}

// Generated scores of a whole tile into shared memory (binary32 patterns, +0 beyond `len`): thread
// q writes elements 32q .. 32q+31, the ones it reads back in the 32-per-thread layout.
__device__ __forceinline__ void stage_tile_scores(float *dst, const TopkSide &s, int row, int t, int64_t rel, int len) {
    const int pos0 = 32 * threadIdx.x;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const int pos = pos0 + 4 * b;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (pos < len) {
            w = s.gen.block((uint32_t)((rel + pos) >> 2), (uint32_t)t, (uint32_t)row);
            if (pos + 1 >= len) w.y = 0u;
            if (pos + 2 >= len) w.z = 0u;
            if (pos + 3 >= len) w.w = 0u;
        }
        *reinterpret_cast<uint4 *>(dst + pos) = w;
    }
}

enum { STATUS_PICK_RANK = 1, STATUS_CAND_OVERFLOW = 2, STATUS_COUNT_MISMATCH = 4 };

// Adds a CTA's shared-memory histogram to the problem's global one and widens the problem's
// record of the non-empty bin range, so that the pick reads and clears only that range.
__device__ __forceinline__ void flush_hist(const uint32_t *h, uint32_t *gh, uint32_t *sel, int lo_word, int hi_word) {
    uint32_t lo = 0xffffffffu, hi = 0u;
    for (uint32_t b = threadIdx.x; b < DIGIT1_BINS; b += blockDim.x) {
        const uint32_t c = h[b];
        if (c) {
            atomicAdd(gh + b, c);
            lo = min(lo, b);
            hi = max(hi, b);
        }
    }
    lo = __reduce_min_sync(0xffffffffu, lo);
    hi = __reduce_max_sync(0xffffffffu, hi);
    if ((threadIdx.x & 31) == 0 && lo != 0xffffffffu) {
        atomicMin(&sel[lo_word], lo);
        atomicMax(&sel[hi_word], hi);
    }
}

// ------------------------------------------------------------------------------------------------
// Block helper: bins[0..nbins) in shared memory, find the bin that holds the rank-th largest
// entry counting from the top bin down.  All threads get (bin, rank inside bin, count above+bin).
// ------------------------------------------------------------------------------------------------
struct PickResult { uint32_t bin, rank_in_bin, count_ge; bool ok; };

template <int NT = THREADS>
__device__ PickResult block_pick(const uint32_t *bins, int nbins, uint32_t rank, uint32_t *scratch /*[NT+4]*/) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = nbins >= NT ? nbins / NT : 1;
    const int active = nbins / per;
    uint32_t mine = 0;
    if (tid < active)
        for (int q = 0; q < per; ++q) mine += bins[tid * per + q];
    // inclusive suffix sum over threads (higher thread = higher bins): shuffles inside a warp,
    // then the totals of the warps above
    uint32_t suf = mine;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const uint32_t up = __shfl_down_sync(0xffffffffu, suf, m);
        if (lane + m < 32) suf += up;
    }
    if (lane == 0) scratch[warp] = suf;  // warp total
    if (tid == 0) scratch[NT + 3] = 0u;  // found flag
    __syncthreads();
    uint32_t above_warps = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w)
        if (w > warp) above_warps += scratch[w];
    const uint32_t suf_incl = suf + above_warps;
    const uint32_t suf_excl = suf_incl - mine;
    if (tid < active && suf_excl < rank && rank <= suf_incl) {
        uint32_t above = suf_excl;
        for (int q = per - 1; q >= 0; --q) {
            uint32_t c = bins[tid * per + q];
            if (above + c >= rank) {
                scratch[NT + 0] = (uint32_t)(tid * per + q);
                scratch[NT + 1] = rank - above;
                scratch[NT + 2] = above + c;
                scratch[NT + 3] = 1u;
                break;
            }
            above += c;
        }
    }
    __syncthreads();
    PickResult r;
    r.bin = scratch[NT + 0];
    r.rank_in_bin = scratch[NT + 1];
    r.count_ge = scratch[NT + 2];
    r.ok = scratch[NT + 3] != 0u;
    __syncthreads();
    return r;
}

// Exclusive prefix sum of one value per thread over the CTA (shuffles inside warps, warp totals in
// shared memory); `total` receives the CTA's sum.  Two barriers.
template <int NT = THREADS>
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t x, uint32_t *warp_tot /*[NT/32]*/, uint32_t &total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = x;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, inc, m);
        if (lane >= m) inc += up;
    }
    __syncthreads();  // warp_tot may still be read from the previous call
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t before = 0;
    total = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) {
        if (w < warp) before += warp_tot[w];
        total += warp_tot[w];
    }
    return before + inc - x;
}

// ------------------------------------------------------------------------------------------------
// Dense path of one problem whose candidates did not fit the buffer even under a 24-bit prefix (huge
// groups of equal magnitudes, e.g. mostly-zero rows): the CTA walks the segment itself.
// ------------------------------------------------------------------------------------------------
template <typename GT, int NT>
__device__ void slow_select(const Params &p, const TopkSide &s, int t, int row, uint32_t *sel, uint32_t *bins,
                            uint32_t *scratch, uint32_t *wa, uint32_t *wb) {
    constexpr int NW = NT / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t seg_beg = __ldg(p.seg_off + t);
    const int64_t n = __ldg(p.seg_off + t + 1) - seg_beg;
    auto value_at = [&](int64_t j) { return fetch1<GT>(s, row, t, seg_beg, j); };
    // U stripes of NT consecutive elements per round: a thread's U loads are in flight together
    constexpr int U = 8;
    static_assert(TILE % (NT * U) == 0, "a round of the dense path must not straddle a tile boundary");
    __shared__ uint32_t cnt_tie[U][NW], cnt_sel[U][NW];
    auto dense_sweep = [&](auto &&use) {   // use(key) for every element of the segment
        for (int64_t j0 = threadIdx.x; j0 < n; j0 += (int64_t)NT * U) {
            uint32_t key[U];
#pragma unroll
            for (int u = 0; u < U; ++u) key[u] = j0 + (int64_t)u * NT < n ? key_of(value_at(j0 + (int64_t)u * NT)) : 0xffffffffu;
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (key[u] != 0xffffffffu) use(key[u]);
        }
    };
    uint32_t rank = sel[SEL_REMAIN];
    uint32_t prefix24;
    const uint32_t flags = sel[SEL_FLAGS];
    if (flags & 2u) {
        prefix24 = sel[SEL_PREFIX];  // found by the dense second-digit pass
    } else {
        const uint32_t b1 = sel[SEL_PREFIX];
        for (int b = threadIdx.x; b < DIGIT1_BINS; b += NT) bins[b] = 0u;
        __syncthreads();
        dense_sweep([&](uint32_t key) { if ((key >> DIGIT1_SHIFT) == b1) atomicAdd(&bins[(key >> 7) & 0xfffu], 1u); });
        __syncthreads();
        const PickResult r2 = block_pick<NT>(bins, DIGIT1_BINS, rank, scratch);
        if (!r2.ok) { if (threadIdx.x == 0) atomicOr(p.status, STATUS_PICK_RANK); return; }
        prefix24 = (b1 << 12) | r2.bin;
        rank = r2.rank_in_bin;
    }
    // last 7 bits
    for (int b = threadIdx.x; b < NT; b += NT) bins[b] = 0u;
    __syncthreads();
    dense_sweep([&](uint32_t key) { if ((key >> 7) == prefix24) atomicAdd(&bins[key & 0x7fu], 1u); });
    __syncthreads();
    const PickResult r = block_pick<NT>(bins, NT, rank, scratch);
    if (!r.ok) { if (threadIdx.x == 0) atomicOr(p.status, STATUS_PICK_RANK); return; }
    const uint32_t T = (prefix24 << 7) | r.bin;
    const uint32_t ties_wanted = r.rank_in_bin;
    __syncthreads();
    if (threadIdx.x == 0) { sel[SEL_THRESH] = T; sel[SEL_TIES] = ties_wanted; }
    // ordered compaction over the dense segment
    const int first_tile = __ldg(p.tile_prefix + t);
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t), k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const int64_t obase = (int64_t)row * p.K + kbeg;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t run_sel = 0, run_tie = 0;
    for (int64_t j0 = 0; j0 < n; j0 += (int64_t)NT * U) {
        if ((j0 % TILE) == 0 && threadIdx.x == 0)   // (a round never straddles a tile boundary)
            s.outbase[(int64_t)row * (p.TT + 1) + first_tile + (int)(j0 / TILE)] = kbeg + run_sel;
        // stripe u holds elements j0 + u*NT .. +NT-1: stripes, and the threads inside one, are in index order
        float val[U];
        uint32_t tb[U], sb[U], tie_rank[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t j = j0 + (int64_t)u * NT + threadIdx.x;
            val[u] = j < n ? value_at(j) : __uint_as_float(0xffffffffu);   // (a pattern no key equals: keys have 31 bits)
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool in = j0 + (int64_t)u * NT + threadIdx.x < n;
            tb[u] = __ballot_sync(0xffffffffu, in && key_of(val[u]) == T);
            if (lane == 0) cnt_tie[u][warp] = __popc(tb[u]);
        }
        __syncthreads();
        uint32_t ties_so_far = run_tie;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool in = j0 + (int64_t)u * NT + threadIdx.x < n;
            const uint32_t key = key_of(val[u]);
            uint32_t before = ties_so_far + __popc(tb[u] & lt_mask), tot = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) { if (w < warp) before += cnt_tie[u][w]; tot += cnt_tie[u][w]; }
            tie_rank[u] = before;
            const bool tie = (tb[u] >> lane) & 1u;
            const bool take = in && (key > T || (tie && before < ties_wanted));
            sb[u] = __ballot_sync(0xffffffffu, take);
            if (lane == 0) cnt_sel[u][warp] = __popc(sb[u]);
            ties_so_far += tot;
        }
        __syncthreads();
        uint32_t sel_so_far = run_sel;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            uint32_t out = sel_so_far + __popc(sb[u] & lt_mask), tot = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) { if (w < warp) out += cnt_sel[u][w]; tot += cnt_sel[u][w]; }
            const bool take = (sb[u] >> lane) & 1u;
            if (take && out >= k) {
                atomicOr(p.status, STATUS_COUNT_MISMATCH);
            } else if (take) {
                const uint32_t flat = (uint32_t)(seg_beg + j0 + (int64_t)u * NT + threadIdx.x);
                s.idx[obase + out] = flat;
                s.val[obase + out] = val[u];
                if (((tb[u] >> lane) & 1u) && tie_rank[u] == ties_wanted - 1) sel[SEL_CUT] = flat;
            }
            sel_so_far += tot;
        }
        run_sel = sel_so_far;
        run_tie = ties_so_far;
        __syncthreads();   // the counters are rewritten by the next round
    }
    if (threadIdx.x == 0 && run_sel != k) atomicOr(p.status, STATUS_COUNT_MISMATCH);
    // downlink: selected entries of the error become +0 (after every read of the segment is done)
    if (s.zero_out) {
        __syncthreads();
        for (uint32_t q = threadIdx.x; q < k; q += NT) s.zero_out[s.idx[obase + q]] = 0.0f;
    }
}

// one launch each (defined in topk_tail.cu)
// src_kind: element type of the selection's source
constexpr int SRC_F32 = 0, SRC_BF16 = 1, SRC_SCORES = 2;
cudaError_t launch_topk_small(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st);
cudaError_t launch_topk_check(const Params &p, const TopkSide &s, cudaStream_t st);
cudaError_t launch_topk_tail(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st, int64_t *launches);
constexpr int64_t TAIL_BIG_CAP = 16384;   // candidate capacity from which a problem's tail gets the larger CTA
cudaError_t configure_topk_tail_kernels();
// seeded random-k draw: the selection on generated scores (defined in topk_kernels.cu)
cudaError_t launch_randk_draw_small(const Params &p, const TopkSide &s, cudaStream_t st, int64_t *launches);
cudaError_t launch_randk_draw(const Params &p, const TopkSide &s, cudaStream_t st, int64_t *launches);

// Limits of the one-CTA-per-problem tail: candidates of one segment that it sweeps, tiles of one
// segment that its shared-memory tables hold.  Beyond either, the same steps run as wide launches.
constexpr int64_t TAIL_MAX_CAND = 1 << 17;
constexpr int TAIL_MAX_TILES = 1024;
inline bool use_fused_tail(const Params &p) { return p.cap_max <= TAIL_MAX_CAND && p.max_seg_tiles <= TAIL_MAX_TILES; }

}  // namespace liec
