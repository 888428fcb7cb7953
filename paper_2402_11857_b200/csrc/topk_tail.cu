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
#include <algorithm>
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
    extern __shared__ __align__(16) unsigned char small_smem[];
    uint32_t *hist = reinterpret_cast<uint32_t *>(small_smem);                               // [DIGIT1_BINS]
    ST *tile_s = reinterpret_cast<ST *>(small_smem + sizeof(uint32_t) * DIGIT1_BINS);        // [TILE]
    __shared__ uint32_t scratch[THREADS + 4];
    __shared__ uint32_t warp_tot[THREADS / 32];
    const int t = __ldg(p.small_seg + blockIdx.x), row = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int64_t seg_beg = __ldg(p.seg_off + t);
    const int n = (int)(__ldg(p.seg_off + t + 1) - seg_beg);
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t), k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    if constexpr (std::is_same<GT, ScoreGen>::value) {
        stage_tile_scores(reinterpret_cast<float *>(tile_s), s, row, t, 0, n);
    } else {
        const int64_t row_beg = (int64_t)row * s.row_stride + seg_beg;
        const ST *src = reinterpret_cast<const ST *>(s.src) + row_beg;
        stage_tile_guarded(tile_s, src, n, (row_beg & (F32 ? 3 : 7)) == 0);
    }

    // thread q owns elements 32q .. 32q+31; it visits them in an order rotated by the lane so that
    // the lanes of a warp hit different banks
    const int pos0 = 32 * threadIdx.x;
    const int valid = min(32, max(0, n - pos0));
    const int rot = F32 ? lane : (lane & ~1);
    auto key_at = [&](int j) -> uint32_t {
        if constexpr (F32) return key_of(tile_s[pos0 + j]);
        else return ((uint32_t)tile_s[pos0 + j] & 0x7fffu) << 16;
    };

    // radix select, most significant digit first: 12 + 12 + 7 key bits (bfloat16 keys have 15 bits: 12 + 3).
    // The wide first digit spreads the entries over many bins (the exponent alone would put nearly
    // all of them into a handful), which keeps the shared-memory atomics from serialising.
    constexpr int LEVELS = F32 ? 3 : 2;
    constexpr int LOW = F32 ? 0 : 16;   // key bits below the last digit (all zero for bfloat16)
    uint32_t prefix = 0u, rank = k;
    bool ok = true;
#pragma unroll
    for (int level = 0; level < LEVELS; ++level) {
        const int bits = level == 0 ? 12 : (F32 ? (level == 1 ? 12 : 7) : 3);
        const int shift = level == 0 ? DIGIT1_SHIFT : (F32 ? (level == 1 ? 7 : 0) : 16);
        const int nbins = bits == 12 ? DIGIT1_BINS : THREADS;   // (block_pick wants at least one bin per thread)
        for (int b = threadIdx.x; b < nbins / 4; b += THREADS) reinterpret_cast<uint4 *>(hist)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();   // (also: the staged tile is complete)
        if (valid > 0) {   // (short segments leave most threads without elements)
            for (int i = 0; i < 32; ++i) {
                const int j = (i + rot) & 31;
                if (j < valid) {
                    const uint32_t key = key_at(j);
                    if ((key >> (shift + bits)) == prefix) atomicAdd(&hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
                }
            }
        }
        __syncthreads();
        const PickResult r = block_pick<THREADS>(hist, nbins, rank, scratch);
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
// CTAs of this kernel are latency-bound chains (sweeps over the candidates with a block-wide pick or
// scan between them), so the launch as a whole is bound by how many of them are resident.  The few
// largest problems (candidate capacity of TAIL_BIG_CAP or more: their CTAs run longest) get 512
// threads in a launch of their own on the context's helper stream (higher priority, so that they
// start first); the many others get 256 threads and bitmaps sized for their own, smaller candidate
// buffers, so that one big CTA and two small ones, or four to five small ones, share an SM.
constexpr int TAIL_THREADS = 256, TAIL_THREADS_BIG = 512;

// Words of one bitmap over `cap` candidates, rounded up to whole rounds of the largest CTA.
static inline int tail_bitmap_words(int64_t cap) {
    const int words = (int)((cap + 31) / 32);
    return (words + TAIL_THREADS_BIG - 1) / TAIL_THREADS_BIG * TAIL_THREADS_BIG;
}

// Problems large_seg[first_problem + blockIdx.x] of every row.
template <typename GT, int NT>
__global__ void __launch_bounds__(NT, 1024 / NT) topk_tail_kernel(const __grid_constant__ Params p, const TopkSide s,
                                                        const int bitmap_words, const int first_problem) {
    constexpr int NW = NT / 32;
    __shared__ __align__(16) uint32_t bins[DIGIT1_BINS];
    __shared__ uint32_t scratch[NT + 4];
    __shared__ uint32_t warp_tot[NW], warp_tot2[NW];
    // per tile: entries above the threshold / equal to it; after the scan over the tiles: first
    // output slot / ties to accept; ties in the tiles before; start of the tile's candidate block
    __shared__ uint32_t t_gt[TAIL_MAX_TILES], t_eq[TAIL_MAX_TILES], t_tb[TAIL_MAX_TILES], t_pos[TAIL_MAX_TILES];
    // one bit per candidate (above the threshold / equal to it) and, per 32-bit word of those
    // bitmaps, the number of set bits in the words before
    extern __shared__ uint32_t tail_smem[];
    uint32_t *gt_bits = tail_smem, *eq_bits = tail_smem + bitmap_words;
    uint32_t *gt_before = tail_smem + 2 * bitmap_words, *eq_before = tail_smem + 3 * bitmap_words;
    const int t = __ldg(p.large_seg + first_problem + blockIdx.x), row = blockIdx.y;
    const int lane = threadIdx.x & 31;
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    // last kernel(s) of a side: the next step starts with "no problem on the regular route yet"
    if (s.spec && blockIdx.x == 0 && row == 0 && threadIdx.x == 0) p.status[STATUS_ANY_REGULAR] = 0;
    const uint32_t flags = sel[SEL_FLAGS];
    const bool single = s.spec && sel[SEL_MODE] == 1u;
    const uint32_t cap = (uint32_t)(__ldg(s.cap_off + t + 1) - __ldg(s.cap_off + t));
    const uint32_t k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t);
    const uint32_t ncand = min(sel[SEL_CAND_COUNT], cap);  // (the cursor can run past the buffer when a tile was refused)
    uint32_t prefix = sel[SEL_PREFIX], rank = sel[SEL_REMAIN];
    uint32_t margin = sel[SEL_MARGIN];
    const int first = __ldg(p.tile_prefix + t), ntiles = __ldg(p.tile_prefix + t + 1) - first;
    const uint32_t seg_first = (uint32_t)__ldg(p.seg_off + t);
    for (int q = threadIdx.x; q < ntiles; q += NT) {
        t_pos[q] = s.meta[((int64_t)row * p.TT + first + q) * 4];
        t_gt[q] = 0u;
        t_eq[q] = 0u;
    }
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
    const int64_t cbase = (int64_t)row * s.CAP + __ldg(s.cap_off + t);
    const float *cand = s.cand_val + cbase;
    const uint32_t *cidx = s.cand_idx + cbase;
    auto fail = [&](int bit) { if (threadIdx.x == 0) { atomicOr(p.status, bit); if (s.spec) sel[SEL_GUESS] = 0u; } };
    auto clear_bins = [&](int nb) {
        for (int b = threadIdx.x; b < nb / 4; b += NT) reinterpret_cast<uint4 *>(bins)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
    };

    // Sweeps over the candidates' values: a thread fetches B values (B stripes of NT consecutive
    // candidates) before it uses any, so that the loads are in flight together.
    constexpr int B = 16;
    auto sweep_keys = [&](auto &&use) {   // use(key) for every candidate of this thread
        for (uint32_t q0 = threadIdx.x; q0 < ncand; q0 += NT * B) {
            uint32_t key[B];
#pragma unroll
            for (int u = 0; u < B; ++u) key[u] = q0 + u * NT < ncand ? key_of(cand[q0 + u * NT]) : 0xffffffffu;
#pragma unroll
            for (int u = 0; u < B; ++u)
                if (key[u] != 0xffffffffu) use(key[u]);
        }
    };

    bool refined = (flags & 2u) != 0u;
    if (single) {
        // First digit from the candidates themselves (all entries at or above the guess).  They crowd
        // into the bins just above the guess, where histogram atomics on one address would serialise:
        // count in registers how many reach each of the WIN lowest bins; the bin of the k-th largest
        // is almost always among them.
        constexpr int WIN = 8;
        const uint32_t gbin = sel[SEL_GUESS] >> DIGIT1_SHIFT;
        uint32_t reach[WIN];
#pragma unroll
        for (int r = 0; r < WIN; ++r) reach[r] = 0u;
        sweep_keys([&](uint32_t key) {
            const uint32_t d1 = key >> DIGIT1_SHIFT;
#pragma unroll
            for (int r = 0; r < WIN; ++r) reach[r] += d1 >= gbin + r + 1u ? 1u : 0u;   // entries above bin gbin + r
        });
        if (threadIdx.x < WIN) bins[threadIdx.x] = 0u;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < WIN; ++r) {
            const uint32_t c = __reduce_add_sync(0xffffffffu, reach[r]);
            if (lane == 0 && c) atomicAdd(&bins[r], c);
        }
        __syncthreads();
        // above[r] = entries above bin gbin + r; all ncand entries are at or above bin gbin
        int found = -1;
        uint32_t above_found = 0u;
#pragma unroll
        for (int r = WIN - 1; r >= 0; --r) {
            const uint32_t above = bins[r];
            if (above < k) { found = r; above_found = above; }   // keeps the lowest r with fewer than k entries above it
        }
        __syncthreads();   // bins are reused below
        if (found >= 0) {
            prefix = gbin + (uint32_t)found;
            rank = k - above_found;
        } else {   // the threshold moved up by more than WIN bins: plain histogram
            clear_bins(DIGIT1_BINS);
            sweep_keys([&](uint32_t key) { atomicAdd(&bins[key >> DIGIT1_SHIFT], 1u); });
            __syncthreads();
            const PickResult r1 = block_pick<NT>(bins, DIGIT1_BINS, k, scratch);
            if (!r1.ok) { fail(STATUS_PICK_RANK); return; }
            prefix = r1.bin;
            rank = r1.rank_in_bin;
        }
        refined = false;
    }
    if (!refined) {   // second digit among the entries that share the threshold's first digit
        const uint32_t b1 = prefix;
        clear_bins(DIGIT1_BINS);
        sweep_keys([&](uint32_t key) { if ((key >> DIGIT1_SHIFT) == b1) atomicAdd(&bins[(key >> 7) & 0xfffu], 1u); });
        __syncthreads();
        const PickResult r2 = block_pick<NT>(bins, DIGIT1_BINS, rank, scratch);
        if (!r2.ok) { fail(STATUS_PICK_RANK); return; }
        prefix = (b1 << 12) | r2.bin;
        rank = r2.rank_in_bin;
    }
    clear_bins(NT);   // last 7 bits (block_pick wants at least NT bins; those above 127 stay empty)
    sweep_keys([&](uint32_t key) { if ((key >> 7) == prefix) atomicAdd(&bins[key & 0x7fu], 1u); });
    __syncthreads();
    const PickResult r3 = block_pick<NT>(bins, NT, rank, scratch);
    if (!r3.ok) { fail(STATUS_PICK_RANK); return; }
    const uint32_t T = (prefix << 7) | r3.bin;
    const uint32_t ties_wanted = r3.rank_in_bin;

    // Sweep over the candidates in buffer order (a warp takes 32 consecutive ones = one bitmap word):
    // the two bitmaps, and per tile the number of entries above the threshold and equal to it.
    // The tile of a candidate follows from its index.
    const uint32_t nwords = (ncand + 31) >> 5;
    constexpr int BX = 8;
    for (uint32_t q0 = threadIdx.x & ~31u; q0 < ncand; q0 += NT * BX) {   // (bounds uniform over the warp)
        uint32_t key[BX], tile[BX];
#pragma unroll
        for (int u = 0; u < BX; ++u) {
            const uint32_t q = q0 + u * NT + lane;
            const bool in = q < ncand;
            key[u] = in ? key_of(cand[q]) : 0u;
            tile[u] = in ? (cidx[q] - seg_first) >> 13 : 0xffffffffu;   // TILE = 2^13
        }
#pragma unroll
        for (int u = 0; u < BX; ++u) {
            const uint32_t qw = q0 + u * NT;
            if (qw >= ncand) break;   // (uniform over the warp)
            const bool in = tile[u] != 0xffffffffu;
            const bool gt = in && key[u] > T, eq = in && key[u] == T;
            const uint32_t gb = __ballot_sync(0xffffffffu, gt), eb = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) { gt_bits[qw >> 5] = gb; eq_bits[qw >> 5] = eb; }
            // lanes of the first lane's tile add once; the others (a block boundary inside the word) one by one
            const uint32_t tile0 = __shfl_sync(0xffffffffu, tile[u], 0);
            const uint32_t same = __ballot_sync(0xffffffffu, tile[u] == tile0);
            if (lane == 0 && tile0 < (uint32_t)ntiles) {
                const uint32_t g = __popc(gb & same), e = __popc(eb & same);
                if (g) atomicAdd(&t_gt[tile0], g);
                if (e) atomicAdd(&t_eq[tile0], e);
            }
            if (in && tile[u] != tile0 && tile[u] < (uint32_t)ntiles) {
                if (gt) atomicAdd(&t_gt[tile[u]], 1u);
                if (eq) atomicAdd(&t_eq[tile[u]], 1u);
            }
        }
    }
    for (uint32_t w = nwords + threadIdx.x; w < (uint32_t)bitmap_words; w += NT) { gt_bits[w] = 0u; eq_bits[w] = 0u; }
    __syncthreads();
    // tiles in order: ties accepted per tile (lowest index first) and first output slot
    constexpr int PER = (TAIL_MAX_TILES + NT - 1) / NT;
    bool all_ties;   // every entry equal to the threshold is kept (the usual case: distinct magnitudes)
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
            fail(STATUS_COUNT_MISMATCH);
            return;
        }
        all_ties = ties_total == ties_wanted;
    }
    // set bits in the bitmap words before each word (when every tie is kept, the first bitmap
    // becomes "kept": above the threshold or equal to it)
    {
        const int perw = bitmap_words / NT;
        const int w0 = threadIdx.x * perw;
        uint32_t gsum = 0, esum = 0;
        if (all_ties)
            for (int u = 0; u < perw; ++u) gt_bits[w0 + u] |= eq_bits[w0 + u];
        for (int u = 0; u < perw; ++u) { gsum += __popc(gt_bits[w0 + u]); esum += __popc(eq_bits[w0 + u]); }
        uint32_t tot;
        uint32_t gpre = block_exclusive_scan<NT>(gsum, warp_tot, tot);
        uint32_t epre = block_exclusive_scan<NT>(esum, warp_tot2, tot);
        for (int u = 0; u < perw; ++u) {
            gt_before[w0 + u] = gpre; gpre += __popc(gt_bits[w0 + u]);
            eq_before[w0 + u] = epre; epre += __popc(eq_bits[w0 + u]);
        }
    }
    __syncthreads();
    // Ordered compaction, candidate-parallel: the slot of a kept candidate is its tile's first slot
    // plus the kept candidates before it in its tile's block (blocks are contiguous and in index
    // order; ties are accepted lowest index first, so the accepted ones before it number
    // min(ties before it in the block, ties accepted in the tile)).
    const int64_t obase = (int64_t)row * p.K + kbeg;
    if (all_ties) {
        // the slot of a kept candidate = (its tile's first slot - kept candidates before the tile's block)
        // + kept candidates before it in the buffer
        for (int q = threadIdx.x; q < ntiles; q += NT) {
            const uint32_t pb = t_pos[q], pw = pb >> 5;
            t_gt[q] -= gt_before[pw] + __popc(gt_bits[pw] & ((1u << (pb & 31u)) - 1u));
        }
        __syncthreads();
        for (uint32_t q0 = threadIdx.x; q0 < ncand; q0 += NT * BX) {
            uint32_t idx[BX];
            float val[BX];
#pragma unroll
            for (int u = 0; u < BX; ++u) {
                const uint32_t q = q0 + u * NT;
                idx[u] = q < ncand ? cidx[q] : 0xffffffffu;
                val[u] = q < ncand ? cand[q] : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < BX; ++u) {
                const uint32_t q = q0 + u * NT;
                if (q >= ncand) break;
                const uint32_t w = q >> 5, bit = q & 31u, kw = gt_bits[w];
                if (!((kw >> bit) & 1u)) continue;
                const uint32_t tile = (idx[u] - seg_first) >> 13;
                if (tile >= (uint32_t)ntiles) continue;
                const uint32_t out = t_gt[tile] + gt_before[w] + __popc(kw & ((1u << bit) - 1u));   // < k by the scan above
                s.idx[obase + out] = idx[u];
                s.val[obase + out] = val[u];
                if (s.zero_out) s.zero_out[idx[u]] = 0.0f;
                if ((eq_bits[w] >> bit) & 1u) {   // the last tie (all are kept): the one with ties_wanted - 1 ties before it
                    const uint32_t pb = t_pos[tile], pw = pb >> 5;
                    const uint32_t e_in_block = eq_before[w] + __popc(eq_bits[w] & ((1u << bit) - 1u)) -
                                                (eq_before[pw] + __popc(eq_bits[pw] & ((1u << (pb & 31u)) - 1u)));
                    if (t_tb[tile] + e_in_block + 1u == ties_wanted) sel[SEL_CUT] = idx[u];
                }
            }
        }
    } else
    for (uint32_t q0 = threadIdx.x; q0 < ncand; q0 += NT * BX) {
        uint32_t idx[BX];
        float val[BX];
#pragma unroll
        for (int u = 0; u < BX; ++u) {   // (all of them: most candidates are kept)
            const uint32_t q = q0 + u * NT;
            idx[u] = q < ncand ? cidx[q] : 0xffffffffu;
            val[u] = q < ncand ? cand[q] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < BX; ++u) {
            const uint32_t q = q0 + u * NT;
            if (q >= ncand) break;
            const uint32_t w = q >> 5, below = (1u << (q & 31u)) - 1u;
            const uint32_t gw = gt_bits[w], ew = eq_bits[w];
            const bool gt = (gw >> (q & 31u)) & 1u, eq = (ew >> (q & 31u)) & 1u;
            if (!gt && !eq) continue;
            const uint32_t tile = (idx[u] - seg_first) >> 13;
            if (tile >= (uint32_t)ntiles) continue;   // (an index outside the segment cannot come out of the filter)
            const uint32_t pb = t_pos[tile], pw = pb >> 5, pbelow = (1u << (pb & 31u)) - 1u;
            const uint32_t g_in_block = gt_before[w] + __popc(gw & below) - (gt_before[pw] + __popc(gt_bits[pw] & pbelow));
            const uint32_t e_in_block = eq_before[w] + __popc(ew & below) - (eq_before[pw] + __popc(eq_bits[pw] & pbelow));
            const uint32_t allowed = t_eq[tile];
            if (eq && e_in_block >= allowed) continue;   // a tie beyond the accepted ones
            const uint32_t out = t_gt[tile] + g_in_block + min(e_in_block, allowed);   // < k by the scan above
            s.idx[obase + out] = idx[u];
            s.val[obase + out] = val[u];
            if (s.zero_out) s.zero_out[idx[u]] = 0.0f;
            if (eq && t_tb[tile] + e_in_block + 1u == ties_wanted) sel[SEL_CUT] = idx[u];
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
constexpr size_t SMALL_SMEM_F32 = sizeof(uint32_t) * DIGIT1_BINS + sizeof(float) * TILE;
constexpr size_t SMALL_SMEM_BF16 = sizeof(uint32_t) * DIGIT1_BINS + sizeof(unsigned short) * TILE;

cudaError_t launch_topk_small(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st) {
    const dim3 grid(p.n_small, s.R);
    if (src_kind == SRC_BF16) topk_small_kernel<__nv_bfloat16><<<grid, THREADS, SMALL_SMEM_BF16, st>>>(p, s);
    else if (src_kind == SRC_SCORES) topk_small_kernel<ScoreGen><<<grid, THREADS, SMALL_SMEM_F32, st>>>(p, s);
    else topk_small_kernel<float><<<grid, THREADS, SMALL_SMEM_F32, st>>>(p, s);
    return cudaGetLastError();
}

cudaError_t launch_topk_check(const Params &p, const TopkSide &s, cudaStream_t st) {
    topk_check_kernel<<<dim3((p.T + 127) / 128, s.R), 128, 0, st>>>(p, s);
    return cudaGetLastError();
}

template <int NT>
static cudaError_t launch_tail_part(const Params &p, const TopkSide &s, int src_kind, int first, int count, int64_t cap,
                                    cudaStream_t st) {
    const dim3 grid(count, s.R);
    const int words = tail_bitmap_words(cap);
    const size_t smem = sizeof(uint32_t) * 4 * (size_t)words;
    if (src_kind == SRC_BF16) topk_tail_kernel<__nv_bfloat16, NT><<<grid, NT, smem, st>>>(p, s, words, first);
    else if (src_kind == SRC_SCORES) topk_tail_kernel<ScoreGen, NT><<<grid, NT, smem, st>>>(p, s, words, first);
    else topk_tail_kernel<float, NT><<<grid, NT, smem, st>>>(p, s, words, first);
    return cudaGetLastError();
}

// Two concurrent launches when the context has a helper stream and some problems are big: those
// (first in large_seg) on the helper stream, forked from and joined to `st` by events, the others
// on `st`; otherwise one launch on `st`.
cudaError_t launch_topk_tail(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st, int64_t *launches) {
    // at most one big problem per SM: a second one would wait behind the first
    const int n_big = p.tail_stream ? std::min(p.n_big, p.num_sms / s.R) : 0;
    cudaError_t e = cudaSuccess;
    if (n_big > 0) {
        cudaStream_t side = static_cast<cudaStream_t>(p.tail_stream);
        cudaEvent_t fork = static_cast<cudaEvent_t>(p.tail_fork), join = static_cast<cudaEvent_t>(p.tail_join);
        if ((e = cudaEventRecord(fork, st)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(side, fork, 0)) != cudaSuccess) return e;
        if ((e = launch_tail_part<TAIL_THREADS_BIG>(p, s, src_kind, 0, n_big, p.cap_max, side)) != cudaSuccess) return e;
        ++*launches;
        if ((e = cudaEventRecord(join, side)) != cudaSuccess) return e;
    }
    if (p.n_large > n_big) {
        // (big problems that found no SM of their own stay in this launch, which then sizes its bitmaps for them)
        const int64_t cap = n_big == p.n_big ? p.cap_rest_max : p.cap_max;
        if ((e = launch_tail_part<TAIL_THREADS>(p, s, src_kind, n_big, p.n_large - n_big, cap, st)) != cudaSuccess) return e;
        ++*launches;
    }
    if (n_big > 0) e = cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(p.tail_join), 0);
    return e;
}

// Opt-in shared memory sizes of the kernels in this file (once per device).
cudaError_t configure_topk_tail_kernels() {
    const int tail_max = (int)(sizeof(uint32_t) * 4 * ((TAIL_MAX_CAND + 31) / 32 + TAIL_THREADS_BIG));
    const void *tails[] = {(const void *)topk_tail_kernel<float, TAIL_THREADS>, (const void *)topk_tail_kernel<__nv_bfloat16, TAIL_THREADS>,
                           (const void *)topk_tail_kernel<ScoreGen, TAIL_THREADS>, (const void *)topk_tail_kernel<float, TAIL_THREADS_BIG>,
                           (const void *)topk_tail_kernel<__nv_bfloat16, TAIL_THREADS_BIG>, (const void *)topk_tail_kernel<ScoreGen, TAIL_THREADS_BIG>};
    cudaError_t e = cudaSuccess;
    for (const void *k : tails)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, tail_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_small_kernel<ScoreGen>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMALL_SMEM_F32);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_small_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMALL_SMEM_F32);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(topk_small_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMALL_SMEM_BF16);
    return e;
}

}  // namespace liec
