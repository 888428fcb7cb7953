// Top-k (Def. 2), the per-problem kernels that finish a selection on one side of the iteration:
//
//   topk_small_kernel  segments of a single tile (n_t <= TILE): one CTA stages the segment in shared
//                      memory and does the whole selection there (radix select on the 31-bit
//                      magnitude key, ties to the lower index, ordered output).  No guess, no
//                      candidate buffer, no other kernel touches these problems.
//   topk_check_kernel  uplink, after the pass that collected candidates with last step's guess:
//                      decides per problem whether the guess held (at least k candidates, buffer
//                      not exceeded) and adapts how far below the threshold the next guess sits.
//   topk_tail_kernel   segments of several tiles, one CTA per problem, on the problem's candidates
//                      (a contiguous region of the candidate buffer, a few per cent of the segment):
//                      remaining key digits -> exact threshold and number of ties to accept ->
//                      per-tile counts -> output offsets -> ordered compaction into (index, value).
//                      Replaces a chain of seven small launches; nothing waits on another CTA.
#include <type_traits>

#include "device_common.cuh"
#include "kernels.h"
#include "topk_common.cuh"

namespace liec {

// ------------------------------------------------------------------------------------------------
// Single-tile segments: grid (n_small, rows).
// ------------------------------------------------------------------------------------------------
template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_small_kernel(const __grid_constant__ Params p, const TopkSide s) {
    constexpr bool F32 = sizeof(GT) == 4;
    using ST = typename std::conditional<F32, float, unsigned short>::type;
    __shared__ __align__(16) ST tile_s[TILE];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t scratch[THREADS + 4];
    __shared__ uint32_t warp_tot[THREADS / 32];
    const int t = __ldg(p.small_seg + blockIdx.x), row = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int64_t seg_beg = __ldg(p.seg_off + t);
    const int n = (int)(__ldg(p.seg_off + t + 1) - seg_beg);
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t), k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const int64_t row_beg = (int64_t)row * s.row_stride + seg_beg;
    const ST *src = reinterpret_cast<const ST *>(s.src) + row_beg;
    stage_tile_guarded(tile_s, src, n, (row_beg & (F32 ? 3 : 7)) == 0);
    __syncthreads();

    // thread q owns elements 32q .. 32q+31; it visits them in an order rotated by the lane so that
    // the lanes of a warp hit different banks
    const int pos0 = 32 * threadIdx.x;
    const int valid = min(32, max(0, n - pos0));
    const int rot = F32 ? lane : (lane & ~1);
    auto key_at = [&](int j) -> uint32_t {
        if constexpr (F32) return key_of(tile_s[pos0 + j]);
        else return ((uint32_t)tile_s[pos0 + j] & 0x7fffu) << 16;
    };

    // radix select, most significant digit first (binary32: 8+8+8+7 bits; bfloat16 keys have only 15 bits: 8+7)
    constexpr int LEVELS = F32 ? 4 : 2;
    constexpr int LOW = F32 ? 0 : 16;   // key bits below the last digit (all zero for bfloat16)
    uint32_t prefix = 0u, rank = k;
    bool ok = true;
#pragma unroll
    for (int level = 0; level < LEVELS; ++level) {
        const int bits = (level == LEVELS - 1) ? 7 : 8;
        const int shift = F32 ? (level == 3 ? 0 : 23 - 8 * level) : (level == 0 ? 23 : 16);
        hist[threadIdx.x] = 0u;   // THREADS == 256 bins
        __syncthreads();
        for (int i = 0; i < 32; ++i) {
            const int j = (i + rot) & 31;
            if (j < valid) {
                const uint32_t key = key_at(j);
                if ((key >> (shift + bits)) == prefix) atomicAdd(&hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
            }
        }
        __syncthreads();
        const PickResult r = block_pick<THREADS>(hist, 256, rank, scratch);
        ok = ok && r.ok;
        prefix = (prefix << bits) | r.bin;
        rank = r.rank_in_bin;
    }
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    if (!ok) {  // cannot happen for 1 <= k <= n; never write from an inconsistent state
        if (threadIdx.x == 0) atomicOr(p.status, STATUS_PICK_RANK);
        return;
    }
    const uint32_t T = prefix << LOW;       // threshold key
    const uint32_t ties_wanted = rank;      // entries equal to T to accept, lowest index first

    uint32_t gt_mask = 0u, eq_mask = 0u;
    for (int i = 0; i < 32; ++i) {
        const int j = (i + rot) & 31;
        if (j < valid) {
            const uint32_t key = key_at(j);
            gt_mask |= (key > T ? 1u : 0u) << j;
            eq_mask |= (key == T ? 1u : 0u) << j;
        }
    }
    uint32_t ties_total, sel_total;
    const uint32_t ties_before = block_exclusive_scan<THREADS>((uint32_t)__popc(eq_mask), warp_tot, ties_total);
    uint32_t allowed = ties_before < ties_wanted ? min((uint32_t)__popc(eq_mask), ties_wanted - ties_before) : 0u;
    uint32_t take = gt_mask, eq_rest = eq_mask, last_tie_bit = 32u;
    for (uint32_t a = 0; a < allowed; ++a) {   // the lowest `allowed` ties of this thread
        const int b = __ffs(eq_rest) - 1;
        eq_rest &= eq_rest - 1;
        take |= 1u << b;
        if (ties_before + a + 1u == ties_wanted) last_tie_bit = (uint32_t)b;
    }
    const uint32_t out_before = block_exclusive_scan<THREADS>((uint32_t)__popc(take), warp_tot, sel_total);
    if (sel_total != k) {   // inconsistent: flag, write nothing
        if (threadIdx.x == 0) atomicOr(p.status, STATUS_COUNT_MISMATCH);
        return;
    }
    const int64_t obase = (int64_t)row * p.K + kbeg + out_before;
    const uint32_t flat0 = (uint32_t)seg_beg + pos0;
    uint32_t rest = take, o = 0;
    while (rest) {
        const int b = __ffs(rest) - 1;
        rest &= rest - 1;
        s.idx[obase + o] = flat0 + b;
        if constexpr (F32) s.val[obase + o] = tile_s[pos0 + b];
        else s.val[obase + o] = __uint_as_float((uint32_t)tile_s[pos0 + b] << 16);
        if (s.zero_out) s.zero_out[flat0 + b] = 0.0f;
        ++o;
    }
    if (last_tie_bit < 32u) sel[SEL_CUT] = flat0 + last_tie_bit;
    if (threadIdx.x == 0) {
        sel[SEL_THRESH] = T;
        sel[SEL_TIES] = ties_wanted;
        sel[SEL_ROUTE] = ROUTE_DIRECT;
        s.outbase[(int64_t)row * (p.TT + 1) + __ldg(p.tile_prefix + t)] = kbeg;
    }
}

// ------------------------------------------------------------------------------------------------
// Uplink: did last step's guess hold?  One thread per (segment, row).
// ------------------------------------------------------------------------------------------------
constexpr uint32_t MARGIN_MAX = 12u;

// First-digit bins between a problem's first guess and its threshold's bin: as many as the candidate
// buffer allows if every bin further down held 1.4 times the entries of the one above (a Gaussian
// tail near its 1 % quantile grows about that fast per bin of 1/16 octave).
__device__ __forceinline__ uint32_t default_margin(uint32_t k, uint32_t cap) {
    uint32_t m = 0;
    float room = (float)cap / (2.0f * (float)k);
    while (room >= 1.4f && m < 8u) { room *= (1.0f / 1.4f); ++m; }
    return m < 1u ? 1u : m;
}

__global__ void topk_check_kernel(const __grid_constant__ Params p, const TopkSide s) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x, row = blockIdx.y;
    if (t >= p.T) return;
    if (__ldg(p.tile_prefix + t + 1) - __ldg(p.tile_prefix + t) == 1) return;   // selected directly
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    const uint32_t k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const bool guess = sel[SEL_GUESS] != 0u;
    const bool overflow = sel[SEL_SPEC_FAIL] != 0u;
    const bool held = guess && !overflow && sel[SEL_CAND_COUNT] >= k;
    if (guess && !held) {   // too much let through: halve the margin; too little: widen it
        const uint32_t m = sel[SEL_MARGIN];
        sel[SEL_MARGIN] = overflow ? max(1u, m / 2u) : min(MARGIN_MAX, m + 2u);
    }
    sel[SEL_MODE] = held ? 1u : 0u;
    sel[SEL_FLAGS] = 0u;
    if (!held) {
        sel[SEL_CAND_COUNT] = 0u;
        p.status[STATUS_ANY_REGULAR] = 1;
    }
}

// ------------------------------------------------------------------------------------------------
// Tail: grid (n_large, rows), NT threads.  Largest segments first (the host orders large_seg so).
// ------------------------------------------------------------------------------------------------
constexpr int TAIL_THREADS = 512;

template <typename GT>
__global__ void __launch_bounds__(TAIL_THREADS) topk_tail_kernel(const __grid_constant__ Params p, const TopkSide s) {
    constexpr int NT = TAIL_THREADS, NW = NT / 32;
    __shared__ __align__(16) uint32_t bins[DIGIT1_BINS];
    __shared__ uint32_t scratch[NT + 4];
    __shared__ uint32_t warp_tot[NW], warp_tot2[NW];
    __shared__ uint32_t t_gt[TAIL_MAX_TILES], t_eq[TAIL_MAX_TILES];   // per tile: entries above the threshold / equal to it;
                                                                      // after the scan: first output slot / ties to accept
    __shared__ uint32_t t_tb[TAIL_MAX_TILES];                         // ties in the tiles before
    const int t = __ldg(p.large_seg + blockIdx.x), row = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    // last kernel of a side: the next step starts with "no problem on the regular route yet"
    if (s.spec && blockIdx.x == 0 && row == 0 && threadIdx.x == 0) p.status[STATUS_ANY_REGULAR] = 0;
    const uint32_t flags = sel[SEL_FLAGS];
    const bool single = s.spec && sel[SEL_MODE] == 1u;
    const uint32_t cap = (uint32_t)(__ldg(p.cap_off + t + 1) - __ldg(p.cap_off + t));
    const uint32_t k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t);
    const uint32_t ncand = min(sel[SEL_CAND_COUNT], cap);  // (the cursor can run past the buffer when a tile was refused)
    uint32_t prefix = sel[SEL_PREFIX], rank = sel[SEL_REMAIN];
    uint32_t margin = sel[SEL_MARGIN];
    __syncthreads();   // every thread holds the state before thread 0 starts rewriting it
    if (threadIdx.x == 0) {   // the next step starts from a clean slate
        sel[SEL_CAND_COUNT] = 0u;
        sel[SEL_SPEC_FAIL] = 0u;
    }
    if (flags & 1u) {   // even the 24-bit prefix leaves too many candidates: dense passes over the segment
        slow_select<GT, NT>(p, s, t, row, sel, bins, scratch, warp_tot, warp_tot2);
        if (threadIdx.x == 0) {
            sel[SEL_ROUTE] = ROUTE_SLOW | ((flags & 2u) ? ROUTE_REFINED : 0);
            if (s.spec) sel[SEL_GUESS] = 0u;
        }
        return;
    }
    const int64_t cbase = (int64_t)row * p.CAP + __ldg(p.cap_off + t);
    const float *cand = s.cand_val + cbase;
    auto fail = [&]() { if (threadIdx.x == 0) { atomicOr(p.status, STATUS_PICK_RANK); if (s.spec) sel[SEL_GUESS] = 0u; } };
    auto clear_bins = [&](int nb) {
        for (int b = threadIdx.x; b < nb / 4; b += NT) reinterpret_cast<uint4 *>(bins)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
    };

    bool refined = (flags & 2u) != 0u;
    if (single) {   // first digit from the candidates themselves (all entries at or above the guess)
        clear_bins(DIGIT1_BINS);
        for (uint32_t q = threadIdx.x; q < ncand; q += NT) atomicAdd(&bins[key_of(cand[q]) >> DIGIT1_SHIFT], 1u);
        __syncthreads();
        const PickResult r1 = block_pick<NT>(bins, DIGIT1_BINS, k, scratch);
        if (!r1.ok) { fail(); return; }
        prefix = r1.bin;
        rank = r1.rank_in_bin;
        refined = false;
    }
    if (!refined) {   // second digit among the entries that share the threshold's first digit
        const uint32_t b1 = prefix;
        clear_bins(DIGIT1_BINS);
        for (uint32_t q = threadIdx.x; q < ncand; q += NT) {
            const uint32_t key = key_of(cand[q]);
            if ((key >> DIGIT1_SHIFT) == b1) atomicAdd(&bins[(key >> 7) & 0xfffu], 1u);
        }
        __syncthreads();
        const PickResult r2 = block_pick<NT>(bins, DIGIT1_BINS, rank, scratch);
        if (!r2.ok) { fail(); return; }
        prefix = (b1 << 12) | r2.bin;
        rank = r2.rank_in_bin;
    }
    clear_bins(512);   // last 7 bits (block_pick wants at least NT bins; those above 127 stay empty)
    for (uint32_t q = threadIdx.x; q < ncand; q += NT) {
        const uint32_t key = key_of(cand[q]);
        if ((key >> 7) == prefix) atomicAdd(&bins[key & 0x7fu], 1u);
    }
    __syncthreads();
    const PickResult r3 = block_pick<NT>(bins, NT, rank, scratch);
    if (!r3.ok) { fail(); return; }
    const uint32_t T = (prefix << 7) | r3.bin;
    const uint32_t ties_wanted = r3.rank_in_bin;

    // per tile (one warp each, no barrier between a warp's tiles): entries above T, entries equal to T
    const int first = __ldg(p.tile_prefix + t), ntiles = __ldg(p.tile_prefix + t + 1) - first;
    const uint32_t *meta0 = s.meta + ((int64_t)row * p.TT + first) * 4;
    for (int q = warp; q < ntiles; q += NW) {
        const uint32_t pos = meta0[4 * q], cnt = meta0[4 * q + 1];
        uint32_t g = 0, e = 0;
        for (uint32_t c = lane; c < cnt; c += 32) {
            const uint32_t key = key_of(cand[pos + c]);
            g += key > T ? 1u : 0u;
            e += key == T ? 1u : 0u;
        }
        g = __reduce_add_sync(0xffffffffu, g);
        e = __reduce_add_sync(0xffffffffu, e);
        if (lane == 0) { t_gt[q] = g; t_eq[q] = e; }
    }
    __syncthreads();
    // tiles in order: ties accepted per tile (lowest index first) and first output slot
    constexpr int PER = TAIL_MAX_TILES / NT;
    {
        const int q0 = threadIdx.x * PER;
        uint32_t g[PER], e[PER], esum = 0;
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const bool in = q0 + u < ntiles;
            g[u] = in ? t_gt[q0 + u] : 0u;
            e[u] = in ? t_eq[q0 + u] : 0u;
            esum += e[u];
        }
        uint32_t ties_total, sel_total;
        uint32_t ties_before = block_exclusive_scan<NT>(esum, warp_tot, ties_total);
        uint32_t allowed[PER], mine = 0;
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            allowed[u] = ties_before < ties_wanted ? min(e[u], ties_wanted - ties_before) : 0u;
            ties_before += e[u];
            mine += g[u] + allowed[u];
        }
        uint32_t out = block_exclusive_scan<NT>(mine, warp_tot2, sel_total);
        uint32_t tb = ties_before - esum;
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            if (q0 + u < ntiles) {
                t_gt[q0 + u] = out;
                t_eq[q0 + u] = allowed[u];
                t_tb[q0 + u] = tb;
                s.outbase[(int64_t)row * (p.TT + 1) + first + q0 + u] = kbeg + out;
            }
            out += g[u] + allowed[u];
            tb += e[u];
        }
        if (sel_total != k) {   // (uniform over the CTA) inconsistent selection state: write nothing
            if (threadIdx.x == 0) { atomicOr(p.status, STATUS_COUNT_MISMATCH); if (s.spec) sel[SEL_GUESS] = 0u; }
            return;
        }
    }
    __syncthreads();
    // ordered compaction, one warp per tile
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int64_t obase = (int64_t)row * p.K + kbeg;
    const uint32_t *cidx = s.cand_idx + cbase;
    for (int q = warp; q < ntiles; q += NW) {
        const uint32_t pos = meta0[4 * q], cnt = meta0[4 * q + 1];
        const uint32_t out0 = t_gt[q], allowed = t_eq[q], tb0 = t_tb[q];
        uint32_t run_sel = 0, run_tie = 0;
        for (uint32_t c0 = 0; c0 < cnt; c0 += 32) {
            const uint32_t c = c0 + lane;
            const bool in = c < cnt;
            const float val = in ? cand[pos + c] : 0.0f;
            const uint32_t idx = in ? cidx[pos + c] : 0u;
            const uint32_t key = key_of(val);
            const bool tie = in && key == T;
            const uint32_t tbal = __ballot_sync(0xffffffffu, tie);
            const uint32_t tie_rank = run_tie + __popc(tbal & lt_mask);
            const bool take = in && (key > T || (tie && tie_rank < allowed));
            const uint32_t sbal = __ballot_sync(0xffffffffu, take);
            if (take) {
                const uint32_t out = out0 + run_sel + __popc(sbal & lt_mask);   // < k by the scan above
                s.idx[obase + out] = idx;
                s.val[obase + out] = val;
                if (s.zero_out) s.zero_out[idx] = 0.0f;
                if (tie && tb0 + tie_rank + 1u == ties_wanted) sel[SEL_CUT] = idx;
            }
            run_sel += __popc(sbal);
            run_tie += __popc(tbal);
        }
    }
    if (threadIdx.x == 0) {
        sel[SEL_THRESH] = T;
        sel[SEL_TIES] = ties_wanted;
        sel[SEL_ROUTE] = (single ? ROUTE_SINGLE : 0) | (refined ? ROUTE_REFINED : 0);
        if (s.spec) {   // next step's guess: `margin` first-digit bins below this threshold's bin
            if (margin == 0u) { margin = default_margin(k, cap); sel[SEL_MARGIN] = margin; }
            const uint32_t b1 = T >> DIGIT1_SHIFT;
            sel[SEL_GUESS] = (!refined && b1 > margin) ? (b1 - margin) << DIGIT1_SHIFT : 0u;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
cudaError_t launch_topk_small(const Params &p, const TopkSide &s, bool bf16, cudaStream_t st) {
    const dim3 grid(p.n_small, s.R);
    if (bf16) topk_small_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(p, s);
    else topk_small_kernel<float><<<grid, THREADS, 0, st>>>(p, s);
    return cudaGetLastError();
}

cudaError_t launch_topk_check(const Params &p, const TopkSide &s, cudaStream_t st) {
    topk_check_kernel<<<dim3((p.T + 127) / 128, s.R), 128, 0, st>>>(p, s);
    return cudaGetLastError();
}

cudaError_t launch_topk_tail(const Params &p, const TopkSide &s, bool bf16, cudaStream_t st) {
    const dim3 grid(p.n_large, s.R);
    if (bf16) topk_tail_kernel<__nv_bfloat16><<<grid, TAIL_THREADS, 0, st>>>(p, s);
    else topk_tail_kernel<float><<<grid, TAIL_THREADS, 0, st>>>(p, s);
    return cudaGetLastError();
}

}  // namespace liec
