// Deterministic top-k (Def. 2) per segment: exact radix select on the 31-bit magnitude key,
// ties broken toward the lower index, output (index, value) compacted in ascending index.
//
// One selection "problem" is a (row, segment) pair; the uplink has N rows (the workers'
// gradients), the downlink one row (v, held in the error buffer).  A segment of a single tile is
// selected directly by one CTA (topk_small_kernel) and takes no part in what follows.  Regular
// route per side, for the other segments:
//
//   hist1   dense pass 1: histogram of the first key digit (bits 30..19) per problem
//           (for the downlink after a top-k uplink it is fused into the server pass)
//   pick 1  bin b1 holding the k-th largest key, rank left inside it, exact candidate count
//   hist2_dense + pick 4   only for problems whose bin b1 is too crowded for the candidate
//           buffer: dense second-digit histogram, 24-bit prefix
//   filter  dense pass 2: entries at or above the prefix appended, in index order inside each
//           tile, to the problem's region of the candidate buffer
//   tail    one CTA per problem, on its candidates: remaining digits -> exact threshold key and
//           the number of ties to accept -> per-tile counts -> output offsets -> ordered
//           compaction into (idx, val) (topk_tail_kernel).  When a segment has more candidates or
//           tiles than one CTA is given, the same steps run as wide launches instead:
//           cand_hist + pick (levels 2, 3), count, scan, write, close.  A problem whose candidates do
//           not fit the buffer even under a 24-bit prefix (huge groups of equal keys) is finished in the
//           dense source: by its one CTA in the tail; in the wide form by three tile-parallel kernels of
//           its own (last-digit histogram, per-tile counts, ordered write) that leave at once otherwise.
//
// The uplink first tries a single-pass route: filter with a guess (a lower bound taken from the
// previous step's threshold), check (did the guess hold?), and straight to the tail; a problem whose
// guess fails, or that has none, takes the regular route in the same step.  The result never
// depends on the guess.
//
// Nothing waits on another CTA; cross-CTA order comes from kernel boundaries.
#include <type_traits>

#include "device_common.cuh"
#include "kernels.h"
#include "topk_common.cuh"

namespace liec {

// ------------------------------------------------------------------------------------------------
// hist1: one CTA per (tile, row)
// ------------------------------------------------------------------------------------------------
template <bool FAST>
__device__ __forceinline__ void hist1_count(uint32_t *h, const float (&v)[8][4], int warp, int lane, int len) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (FAST || pos + c < len) atomicAdd(&h[key_of(v[j][c]) >> DIGIT1_SHIFT], 1u);
    }
}

template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_hist1_kernel(const __grid_constant__ Params p, const TopkSide s) {
    __shared__ __align__(16) uint32_t h[DIGIT1_BINS];
    if (s.spec && p.status[STATUS_ANY_REGULAR] == 0) return;  // every problem went the single-pass route
    const int row = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int tile = blockIdx.x; tile < p.TT; tile += gridDim.x) {
        const TileInfo ti = locate_tile(p, tile);
        if (ti.seg_tiles == 1) continue;              // selected directly by one CTA
        uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        if (s.spec && sel[SEL_MODE] != 0u) continue;  // uniform over the CTA
        float v[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) fetch4<GT>(s, row, ti, tile_pos(warp, lane, j), v[j]);
        for (int b = threadIdx.x; b < DIGIT1_BINS / 4; b += THREADS) reinterpret_cast<uint4 *>(h)[b] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
        if (ti.len == TILE) hist1_count<true>(h, v, warp, lane, ti.len);
        else hist1_count<false>(h, v, warp, lane, ti.len);
        __syncthreads();
        flush_hist(h, s.hist + ((int64_t)row * p.T + ti.t) * DIGIT1_BINS, sel, SEL_LO1, SEL_HI1);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// pick: one CTA per (segment, row).  level 1: first digit; 2: second digit; 3: last 7 bits.
// The histogram is cleared for the next use.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS) topk_pick_kernel(const __grid_constant__ Params p, const TopkSide s,
                                                             const int level) {
    __shared__ __align__(16) uint32_t bins[DIGIT1_BINS];
    __shared__ uint32_t scratch[THREADS + 4];
    const int t = blockIdx.x, row = blockIdx.y;
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    if (level == 4 && t == 0 && row == 0 && threadIdx.x == 0) p.status[STATUS_ANY_REFINE + (s.zero_out ? 1 : 0)] = 0;
    if (__ldg(p.tile_prefix + t + 1) - __ldg(p.tile_prefix + t) == 1) return;   // selected directly by one CTA
    // level 1: first digit from the dense histogram (regular route).
    // level 5: first digit from the histogram of the candidates collected with the guess
    //          (uplink single-pass route); checks the guess.
    // level 4: second digit of "refined" problems, after their dense second-digit pass.
    // levels 2, 3: wide form of the finish step (second digit, last 7 bits) from candidate histograms.
    if (level == 5 && sel[SEL_MODE] != 1u) return;
    if (level == 2 && sel[SEL_FLAGS] != 0u) return;
    if (level == 1 && s.spec && sel[SEL_MODE] != 0u) return;
    if (level == 4 && sel[SEL_FLAGS] != 2u) return;
    const bool first = level == 1 || level == 5;
    uint32_t *gh = (first ? s.hist : s.hist2) + ((int64_t)row * p.T + t) * DIGIT1_BINS;
    // only the recorded non-empty range of the histogram is read and cleared
    const int lo_word = first ? SEL_LO1 : SEL_LO2, hi_word = first ? SEL_HI1 : SEL_HI2;
    const uint32_t lo = min(sel[lo_word], (uint32_t)DIGIT1_BINS);
    const uint32_t hi = min(sel[hi_word], (uint32_t)DIGIT1_BINS - 1u);
    for (int b = threadIdx.x; b < DIGIT1_BINS / 4; b += THREADS) reinterpret_cast<uint4 *>(bins)[b] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    for (uint32_t b = lo + threadIdx.x; b <= hi; b += THREADS) {
        const uint32_t c = gh[b];
        if (c) { bins[b] = c; gh[b] = 0u; }
    }
    __syncthreads();
    if (threadIdx.x == 0) { sel[lo_word] = 0xffffffffu; sel[hi_word] = 0u; }
    const uint32_t k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    const uint32_t rank = first ? k : sel[SEL_REMAIN];
    const PickResult r = block_pick(bins, DIGIT1_BINS, rank, scratch);
    if (threadIdx.x != 0) return;
    if (!r.ok) { atomicOr(p.status, STATUS_PICK_RANK); return; }
    if (level == 5) {   // (the check kernel has made sure that there are at least k candidates)
        sel[SEL_PREFIX] = r.bin;
        sel[SEL_REMAIN] = r.rank_in_bin;
        sel[SEL_ABOVE] = r.count_ge - bins[r.bin];
        sel[SEL_NCAND] = sel[SEL_CAND_COUNT];
        return;
    }
    const uint32_t cap = (uint32_t)(__ldg(s.cap_off + t + 1) - __ldg(s.cap_off + t));
    if (level == 2) {
        sel[SEL_PREFIX] = (sel[SEL_PREFIX] << 12) | r.bin;
        sel[SEL_REMAIN] = r.rank_in_bin;
    } else if (level == 3) {
        const uint32_t thresh = (sel[SEL_PREFIX] << 7) | r.bin;
        sel[SEL_THRESH] = thresh;
        sel[SEL_TIES] = r.rank_in_bin;
        if (s.spec) {  // next step's guess: one first-digit bin below this threshold's bin
            const uint32_t b1 = thresh >> DIGIT1_SHIFT;
            sel[SEL_GUESS] = (sel[SEL_FLAGS] == 0u && b1 >= 1u) ? (b1 - 1u) << DIGIT1_SHIFT : 0u;
        }
    } else if (level == 1) {
        sel[SEL_PREFIX] = r.bin;
        sel[SEL_REMAIN] = r.rank_in_bin;
        sel[SEL_NCAND] = r.count_ge;
        sel[SEL_ABOVE] = r.count_ge - bins[r.bin];
        sel[SEL_CAND_COUNT] = 0u;
        // too many entries share the threshold's first digit: look at the second digit first
        sel[SEL_FLAGS] = r.count_ge > cap ? 2u : 0u;
        if (r.count_ge > cap) p.status[STATUS_ANY_REFINE + (s.zero_out ? 1 : 0)] = 1;
    } else {
        const uint32_t ncand = sel[SEL_ABOVE] + r.count_ge;
        sel[SEL_PREFIX] = (sel[SEL_PREFIX] << 12) | r.bin;
        sel[SEL_REMAIN] = r.rank_in_bin;
        sel[SEL_NCAND] = ncand;
        if (ncand > cap) {  // still too many (huge groups of equal keys): no candidates, finished in the dense source
            sel[SEL_FLAGS] = 3u;
            sel[SEL_GUESS] = 0u;
            p.status[STATUS_ANY_DENSE + (s.zero_out ? 1 : 0)] = 1;
        }
    }
}

// Dense second-digit pass for refined problems only: histogram of key bits 18..7 over the
// entries whose first digit equals the threshold's.  One CTA per (tile, row).
template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_hist2_dense_kernel(const __grid_constant__ Params p, const TopkSide s) {
    __shared__ uint32_t h[DIGIT1_BINS];
    // usually no problem on this side is refined: a small grid that leaves after one load
    if (p.status[STATUS_ANY_REFINE + (s.zero_out ? 1 : 0)] == 0) return;
    const int row = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // a CTA owns a run of consecutive tiles and keeps one shared histogram per segment of the run:
    // it is flushed when the segment changes and at the end, not after every tile
    const int chunk = (p.TT + gridDim.x - 1) / gridDim.x;
    const int tile_end = min(p.TT, ((int)blockIdx.x + 1) * chunk);
    int open_t = -1;   // segment whose counts the shared histogram holds (uniform over the CTA)
    auto flush_open = [&]() {
        __syncthreads();
        flush_hist(h, s.hist2 + ((int64_t)row * p.T + open_t) * DIGIT1_BINS, s.sel + ((int64_t)row * p.T + open_t) * SEL_WORDS,
                   SEL_LO2, SEL_HI2);
        __syncthreads();
    };
    for (int tile = blockIdx.x * chunk; tile < tile_end; ++tile) {
        const TileInfo ti = locate_tile(p, tile);
        uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        if (sel[SEL_FLAGS] != 2u) continue;  // uniform over the CTA
        const uint32_t b1 = sel[SEL_PREFIX];
        if (ti.t != open_t) {
            if (open_t >= 0) flush_open();
            for (int b = threadIdx.x; b < DIGIT1_BINS; b += THREADS) h[b] = 0u;
            __syncthreads();
            open_t = ti.t;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pos = tile_pos(warp, lane, j);
            float v[4];
            fetch4<GT>(s, row, ti, pos, v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t key = key_of(v[c]);
                if (pos + c < ti.len && (key >> DIGIT1_SHIFT) == b1) atomicAdd(&h[(key >> 7) & 0xfffu], 1u);
            }
        }
    }
    if (open_t >= 0) flush_open();
}

// ------------------------------------------------------------------------------------------------
// filter: one CTA per (tile, row); ordered append of candidates
// ------------------------------------------------------------------------------------------------
// ------------------------------------------------------------------------------------------------
// filter: the tile is staged through shared memory by one TMA bulk copy.
//
// SPEC = true: the uplink's first pass of a step, for problems that have a guess; candidates are
// the entries at or above the guess.  SPEC = false: the regular pass (threshold bin known from the
// histogram); on the uplink it only serves the problems that did not take the single-pass route.
//
// With the tile in shared memory a thread can own 32 CONSECUTIVE elements (16-byte chunks read in
// a lane-rotated order that keeps the banks conflict-free), so its 32-bit candidate mask is
// already in index order and the position of every candidate follows from one exclusive scan of
// the per-thread counts.  A candidate is an entry whose magnitude is at least `low` (a magnitude
// bit pattern used as a float: for finite values the order is the same).  Ragged or misaligned
// tiles are copied with guarded loads instead of the bulk copy and then take the same path.
// ------------------------------------------------------------------------------------------------
// GT = float or __nv_bfloat16: the element type of the source (bf16 tiles are half the bytes; a
// thread's 32 elements are then four 16-byte chunks instead of eight).
template <typename GT, bool SPEC>
__global__ void __launch_bounds__(THREADS) topk_filter_tma_kernel(const __grid_constant__ Params p, const TopkSide s) {
    constexpr bool F32 = sizeof(GT) == 4;
    constexpr bool GEN = std::is_same<GT, ScoreGen>::value;                  // generated scores: nothing to copy
    using ST = typename std::conditional<F32, float, unsigned short>::type;  // storage type of one element
    constexpr int ALIGN_MASK = F32 ? 3 : 7;                                  // elements per 16 bytes, minus one
    __shared__ __align__(128) ST tile_s[TILE];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t warp_tot[8];
    __shared__ uint32_t tile_base;
    if (!SPEC && s.spec && p.status[STATUS_ANY_REGULAR] == 0) return;
    const int row = blockIdx.y, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t phase = 0;
    for (int tile = blockIdx.x; tile < p.TT; tile += gridDim.x) {
        const TileInfo ti = locate_tile(p, tile);
        if (ti.seg_tiles == 1) continue;   // selected directly by one CTA
        uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        float low;
        if (SPEC) {
            // (uniform over the CTA, like every `continue` before the barriers: no kernel writes, in the
            // launch in which it runs, a word that it branches on; a guess that fails is recorded in
            // SEL_SPEC_FAIL, which only later launches read)
            const uint32_t guess = sel[SEL_GUESS];
            if (guess == 0u) continue;
            low = __uint_as_float(guess);
        } else {
            if (s.spec && sel[SEL_MODE] != 0u) continue;
            const uint32_t flags = sel[SEL_FLAGS];
            if (flags & 1u) continue;
            low = __uint_as_float(sel[SEL_PREFIX] << (flags == 2u ? 7 : DIGIT1_SHIFT));
        }
        const int64_t row_beg = (int64_t)row * s.row_stride + ti.seg_beg;
        const ST *tile_ptr = GEN ? nullptr : reinterpret_cast<const ST *>(s.src) + row_beg + ti.rel;
        const bool fast = (ti.len == TILE) && (GEN || (row_beg & ALIGN_MASK) == 0);
        if constexpr (GEN) {
            // nothing to stage: the scores are computed in registers below
        } else if (fast) {
            if (threadIdx.x == 0) {
                const uint32_t bytes = TILE * sizeof(ST);
                // (earlier ordinary reads of the buffer are ordered before the copy by the barrier above)
                bulk_copy_g2s(tile_s, tile_ptr, bytes, bytes + p.copy_expect_extra, &bar);
            }
            // bounded wait for the copy (a wait that never ends must not hang the GPU): flag it, give a
            // copy that may still be in flight time to land, and leave without touching any output
            if (!mbar_wait_bounded(&bar, phase, p.copy_wait_limit)) {
                atomicOr(p.status, STATUS_COPY_TIMEOUT);
                mbar_drain(&bar, phase);
                return;
            }
            phase ^= 1u;
        } else {
            stage_tile_guarded(tile_s, tile_ptr, ti.len, (row_beg & ALIGN_MASK) == 0);
            __syncthreads();
        }
        // 32 consecutive elements per thread, chunk order rotated by the lane
        const int pos0 = 32 * threadIdx.x;
        uint32_t mask = 0;
        if constexpr (GEN) {
            // scores are 30-bit integers whose binary32 reading has the same order: compare the bits
            const uint32_t low_bits = __float_as_uint(low);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 w = s.gen.block((uint32_t)((ti.rel + pos0 + 4 * c) >> 2), (uint32_t)ti.t, (uint32_t)row);
                const uint32_t nib = (w.x >= low_bits ? 1u : 0u) | (w.y >= low_bits ? 2u : 0u) |
                                     (w.z >= low_bits ? 4u : 0u) | (w.w >= low_bits ? 8u : 0u);
                mask |= nib << (4 * c);
            }
        } else if constexpr (F32) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const int c = (kk + lane) & 7;
                const float4 q4 = *reinterpret_cast<const float4 *>(&tile_s[pos0 + 4 * c]);
                uint32_t nib = (fabsf(q4.x) >= low ? 1u : 0u) | (fabsf(q4.y) >= low ? 2u : 0u) |
                               (fabsf(q4.z) >= low ? 4u : 0u) | (fabsf(q4.w) >= low ? 8u : 0u);
                mask |= nib << (4 * c);
            }
        } else {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const int c = (kk + (lane >> 1)) & 3;
                const uint4 q4 = *reinterpret_cast<const uint4 *>(&tile_s[pos0 + 8 * c]);
                const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
                uint32_t byte = 0;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    if (fabsf(__uint_as_float(w4[m] << 16)) >= low) byte |= 1u << (2 * m);
                    if (fabsf(__uint_as_float(w4[m] & 0xffff0000u)) >= low) byte |= 2u << (2 * m);
                }
                mask |= byte << (8 * c);
            }
        }
        if (!fast) {  // drop the padding of a ragged tile
            const int valid = ti.len - pos0;
            mask = valid >= 32 ? mask : (valid <= 0 ? 0u : (mask & ((1u << valid) - 1u)));
        }
        uint32_t tile_cnt;
        const uint32_t before = block_exclusive_scan((uint32_t)__popc(mask), warp_tot, tile_cnt);
        if (threadIdx.x == 0) {
            const uint32_t cap = (uint32_t)(__ldg(s.cap_off + ti.t + 1) - __ldg(s.cap_off + ti.t));
            uint32_t at = tile_cnt ? atomicAdd(&sel[SEL_CAND_COUNT], tile_cnt) : 0u;
            if (at + tile_cnt > cap) {
                if (SPEC) {  // the guess lets too much through: this problem takes the regular route
                    sel[SEL_SPEC_FAIL] = 1u;
                    p.status[STATUS_ANY_REGULAR] = 1;
                } else {
                    atomicOr(p.status, STATUS_CAND_OVERFLOW);
                }
                at = 0xffffffffu;
            }
            tile_base = at;
            uint32_t *m = s.meta + ((int64_t)row * p.TT + tile) * 4;
            m[0] = at == 0xffffffffu ? 0u : at;
            m[1] = at == 0xffffffffu ? 0u : tile_cnt;
        }
        __syncthreads();
        const uint32_t base_now = tile_base;
        if (base_now != 0xffffffffu && mask != 0u) {
            const int64_t cbase = (int64_t)row * s.CAP + __ldg(s.cap_off + ti.t) + base_now + before;
            const uint32_t flat0 = (uint32_t)(ti.seg_beg + ti.rel) + pos0;
            uint32_t rest = mask, o = 0;
            while (rest) {  // candidates are rare: usually zero or one iteration
                const int b = __ffs(rest) - 1;
                rest &= rest - 1;
                s.cand_idx[cbase + o] = flat0 + b;
                if constexpr (GEN) s.cand_val[cbase + o] = fetch1<GT>(s, row, ti.t, ti.seg_beg, ti.rel + pos0 + b);   // (candidates are rare: recomputed)
                else if constexpr (F32) s.cand_val[cbase + o] = tile_s[pos0 + b];
                else s.cand_val[cbase + o] = __uint_as_float((uint32_t)tile_s[pos0 + b] << 16);
                ++o;
            }
        }
        __syncthreads();  // the tile buffer, warp_tot and tile_base are rewritten by the next tile
    }
}

// ------------------------------------------------------------------------------------------------
// candidate passes: one CTA per (tile, row) walks that tile's block of the candidate buffer
// ------------------------------------------------------------------------------------------------
struct CandBlock { int64_t base; uint32_t cnt; int t, seg_tiles; uint32_t *sel; uint32_t *meta; uint4 m; bool skip; };

// (the tile's metadata does not depend on its segment: it is fetched beside the segment lookup, not after it)
__device__ __forceinline__ CandBlock cand_block(const Params &p, const TopkSide &s, int tile, int row) {
    CandBlock cb;
    cb.meta = s.meta + ((int64_t)row * p.TT + tile) * 4;
    cb.m = *reinterpret_cast<const uint4 *>(cb.meta);   // pos, cnt, and what the count / scan kernels left
    const TileInfo ti = locate_tile(p, tile);
    cb.t = ti.t;
    cb.seg_tiles = ti.seg_tiles;
    cb.sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
    const uint32_t flags = cb.sel[SEL_FLAGS];
    const int64_t cap0 = __ldg(s.cap_off + ti.t);
    cb.skip = (flags & 1u) != 0u || ti.seg_tiles == 1;
    cb.cnt = cb.skip ? 0u : cb.m.y;
    cb.base = (int64_t)row * s.CAP + cap0 + cb.m.x;
    return cb;
}

// The candidate passes give one warp to every tile block (8 tiles per CTA): blocks are small
// (about 1.4 % of a tile) and warps need no block-wide synchronisation.
// Histograms over candidates, one warp per tile block; lanes holding the same digit add once
// (match + leader).  level 0: first digit, problems on the single-pass route.  level 1 and 2 are
// the wide form of the finish step, for segments whose candidates are too many for one CTA:
// level 1 = second digit of the candidates whose first digit is the threshold's, level 2 = last
// 7 bits of the candidates under the 24-bit prefix.
__global__ void __launch_bounds__(THREADS) topk_cand_hist_kernel(const __grid_constant__ Params p, const TopkSide s,
                                                                  const int level, const int reps) {
    const int row = blockIdx.y, lane = threadIdx.x & 31;
    // a CTA owns 8 * reps consecutive tiles; warp w takes tiles tile0 + w, tile0 + 8 + w, ...
    const int tile0 = blockIdx.x * 8 * reps;
    const int lo_word = level == 0 ? SEL_LO1 : SEL_LO2, hi_word = level == 0 ? SEL_HI1 : SEL_HI2;
    for (int rep = 0; rep < reps; ++rep) {
        const int tile = tile0 + rep * 8 + (threadIdx.x >> 5);
        bool active = tile < p.TT;
        CandBlock cb;
        uint32_t prefix = 0;
        if (active) {
            cb = cand_block(p, s, tile, row);
            const uint32_t flags = cb.sel[SEL_FLAGS];
            active = !cb.skip && cb.seg_tiles < LONG_SEG_TILES &&   // (long segments: topk_cand_hist_long_kernel)
                     !(level == 0 && cb.sel[SEL_MODE] != 1u) && !(level == 1 && flags != 0u);
            prefix = cb.sel[SEL_PREFIX];
        }
        uint32_t lo = 0xffffffffu, hi = 0u;
        if (active) {
            uint32_t *gh = (level == 0 ? s.hist : s.hist2) + ((int64_t)row * p.T + cb.t) * DIGIT1_BINS;
            for (uint32_t c0 = 0; c0 < cb.cnt; c0 += 32) {
                const uint32_t q = c0 + lane;
                uint32_t digit = 0xffffffffu;  // lanes with nothing to add
                if (q < cb.cnt) {
                    const uint32_t key = key_of(s.cand_val[cb.base + q]);
                    if (level == 0) digit = key >> DIGIT1_SHIFT;
                    else if (level == 1) { if ((key >> DIGIT1_SHIFT) == prefix) digit = (key >> 7) & 0xfffu; }
                    else if ((key >> 7) == prefix) digit = key & 0x7fu;
                }
                const uint32_t same = __match_any_sync(0xffffffffu, digit);
                if (digit != 0xffffffffu) {
                    if (lane == __ffs(same) - 1) atomicAdd(gh + digit, (uint32_t)__popc(same));
                    lo = min(lo, digit);
                    hi = max(hi, digit);
                }
            }
            lo = __reduce_min_sync(0xffffffffu, lo);
            hi = __reduce_max_sync(0xffffffffu, hi);
            if (lane == 0 && lo != 0xffffffffu) {
                atomicMin(&cb.sel[lo_word], lo);
                atomicMax(&cb.sel[hi_word], hi);
            }
        }
    }
}

// The same histograms for the long segments (LONG_SEG_TILES tiles or more: flat vectors, an embedding
// matrix).  A problem's candidates are one contiguous region of the buffer, whatever tile they came
// from, and a histogram does not care about their order: a CTA takes `batches` runs of 8192
// consecutive candidates; a thread fetches 32 of a run with eight 128-bit loads before it uses any,
// counts in shared memory, and the CTA adds its non-empty bins to the problem's histogram once (with
// many small CTAs those additions, thousands of CTAs on the same 4096 words, are what the launch
// waits for: hence several runs per CTA where there are tens of millions of candidates).
// Grid (n_long * chunks, rows); chunks past the problem's candidate count leave at once.
constexpr int CAND_RUN = THREADS * 32;
__global__ void __launch_bounds__(THREADS) topk_cand_hist_long_kernel(const __grid_constant__ Params p, const TopkSide s,
                                                                       const int level, const int chunks, const int batches) {
    __shared__ uint32_t h[DIGIT1_BINS];
    const int t = __ldg(p.large_seg + blockIdx.x / chunks), row = blockIdx.y;
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    const uint32_t flags = sel[SEL_FLAGS];
    if ((flags & 1u) || (level == 0 && sel[SEL_MODE] != 1u) || (level == 1 && flags != 0u)) return;   // (uniform over the CTA)
    const uint32_t cap = (uint32_t)(__ldg(s.cap_off + t + 1) - __ldg(s.cap_off + t));
    const uint32_t ncand = min(sel[SEL_CAND_COUNT], cap);
    // positions are counted from the 16-byte boundary at or before the region's first candidate
    const int64_t base = (int64_t)row * s.CAP + __ldg(s.cap_off + t);
    const uint32_t lead = (uint32_t)(base & 3);
    const float *al = s.cand_val + (base - lead);
    const uint32_t end = lead + ncand;
    const uint32_t c0 = (uint32_t)(blockIdx.x % chunks) * (uint32_t)(batches * CAND_RUN);
    if (c0 >= end) return;
    const uint32_t prefix = sel[SEL_PREFIX];
    for (int b = threadIdx.x; b < DIGIT1_BINS / 4; b += THREADS) reinterpret_cast<uint4 *>(h)[b] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    // First digit: the candidates are the entries at or above the guess and crowd into the few bins
    // from the guess's upwards, where atomics on one address would serialise; those bins are counted in
    // registers (near[r]: first digit = guess's bin + r) and only the rare entries further up go to
    // shared memory one by one.
    constexpr int NEAR = 8;
    const uint32_t gbin = sel[SEL_GUESS] >> DIGIT1_SHIFT;
    uint32_t near[NEAR];
#pragma unroll
    for (int r = 0; r < NEAR; ++r) near[r] = 0u;
#pragma unroll 1
    for (int batch = 0; batch < batches; ++batch) {
        const uint32_t r0 = c0 + (uint32_t)(batch * CAND_RUN);
        if (r0 >= end) break;   // (uniform over the CTA)
        uint32_t key[8][4];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = r0 + (uint32_t)(u * THREADS + threadIdx.x) * 4u;
            if (i >= lead && i + 3u < end) {
                const uint4 q = *reinterpret_cast<const uint4 *>(al + i);
                key[u][0] = q.x & 0x7fffffffu; key[u][1] = q.y & 0x7fffffffu;
                key[u][2] = q.z & 0x7fffffffu; key[u][3] = q.w & 0x7fffffffu;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) key[u][j] = (i + j >= lead && i + j < end) ? key_of(al[i + j]) : 0xffffffffu;
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t key1 = key[u][j];
                if (key1 == 0xffffffffu) continue;
                if (level == 0) {
                    const uint32_t rel = (key1 >> DIGIT1_SHIFT) - gbin;
                    if (rel < (uint32_t)NEAR) {
#pragma unroll
                        for (int r = 0; r < NEAR; ++r) near[r] += rel == (uint32_t)r ? 1u : 0u;
                    } else {
                        atomicAdd(&h[key1 >> DIGIT1_SHIFT], 1u);
                    }
                } else if (level == 1) {
                    if ((key1 >> DIGIT1_SHIFT) == prefix) atomicAdd(&h[(key1 >> 7) & 0xfffu], 1u);
                } else if ((key1 >> 7) == prefix) {
                    atomicAdd(&h[key1 & 0x7fu], 1u);
                }
            }
        }
    }
    if (level == 0) {
#pragma unroll
        for (int r = 0; r < NEAR; ++r) {
            const uint32_t c = __reduce_add_sync(0xffffffffu, near[r]);
            if ((threadIdx.x & 31) == 0 && c && gbin + r < (uint32_t)DIGIT1_BINS) atomicAdd(&h[gbin + r], c);
        }
    }
    __syncthreads();
    flush_hist(h, (level == 0 ? s.hist : s.hist2) + ((int64_t)row * p.T + t) * DIGIT1_BINS, sel,
               level == 0 ? SEL_LO1 : SEL_LO2, level == 0 ? SEL_HI1 : SEL_HI2);
}

__global__ void __launch_bounds__(THREADS) topk_count_kernel(const __grid_constant__ Params p, const TopkSide s) {
    const int row = blockIdx.y, lane = threadIdx.x & 31;
    const int tile = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (tile >= p.TT) return;
    const CandBlock cb = cand_block(p, s, tile, row);
    const uint32_t T = cb.sel[SEL_THRESH];
    if (cb.skip) return;
    uint32_t g = 0, e = 0;
    for (uint32_t q0 = lane; q0 < cb.cnt; q0 += 128) {   // four stripes of 32 candidates in flight
        uint32_t key[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) key[u] = q0 + 32 * u < cb.cnt ? key_of(s.cand_val[cb.base + q0 + 32 * u]) : 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool in = q0 + 32 * u < cb.cnt;
            g += in && key[u] > T ? 1u : 0u;
            e += in && key[u] == T ? 1u : 0u;
        }
    }
    g = __reduce_add_sync(0xffffffffu, g);
    e = __reduce_add_sync(0xffffffffu, e);
    if (lane == 0) { cb.meta[2] = g; cb.meta[3] = e; }
}

// scan: one CTA per (segment, row); tiles of the segment in order
// A CTA takes one run of SCAN_PART consecutive tiles of one problem (PER tiles per thread, their
// metadata loads in flight together).  Segments longer than one run are scanned in two launches:
// phase 0 leaves each run's sums of the per-tile counts, phase 1 starts every run from the sums of
// the runs before it (what the ties before a run were allowed follows from their number alone: ties
// are accepted in index order until ties_wanted are).  Grid (T * scan_parts, rows).
__global__ void __launch_bounds__(THREADS) topk_scan_kernel(const __grid_constant__ Params p, const TopkSide s, const int phase) {
    __shared__ uint32_t warp_tot[8];
    constexpr int PER = SCAN_PART / THREADS;
    const int t = blockIdx.x / p.scan_parts, part = blockIdx.x % p.scan_parts, row = blockIdx.y;
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    const int first = __ldg(p.tile_prefix + t), ntiles = __ldg(p.tile_prefix + t + 1) - first;
    if (ntiles == 1) return;   // selected directly by one CTA
    const int c0 = part * SCAN_PART;
    if (c0 >= ntiles) return;
    uint32_t *run_sums = s.scan_parts + (((int64_t)row * p.T + t) * p.scan_parts) * 2;
    const int q0 = c0 + threadIdx.x * PER;
    uint32_t g[PER], e[PER], gsum = 0, esum = 0;
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        const bool in = q0 + u < ntiles;
        const uint4 m = *reinterpret_cast<const uint4 *>(s.meta + ((int64_t)row * p.TT + first + (in ? q0 + u : 0)) * 4);
        g[u] = in ? m.z : 0u;
        e[u] = in ? m.w : 0u;
        gsum += g[u];
        esum += e[u];
    }
    if (phase == 0) {
        uint32_t g_total, e_total;
        block_exclusive_scan(gsum, warp_tot, g_total);
        block_exclusive_scan(esum, warp_tot, e_total);
        if (threadIdx.x == 0) { run_sums[2 * part] = g_total; run_sums[2 * part + 1] = e_total; }
        return;
    }
    const uint32_t ties_wanted = sel[SEL_TIES];
    const uint32_t kbeg = (uint32_t)__ldg(p.k_off + t), k = (uint32_t)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    uint32_t g_before = 0, carry_ties = 0;  // over the runs before this one (uniform over the CTA)
    for (int j = 0; j < part; ++j) { g_before += run_sums[2 * j]; carry_ties += run_sums[2 * j + 1]; }
    const uint32_t carry_sel = g_before + min(carry_ties, ties_wanted);
    uint32_t ties_total, sel_total;
    uint32_t ties_before = carry_ties + block_exclusive_scan(esum, warp_tot, ties_total);
    uint32_t allowed[PER], mine = 0;
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        allowed[u] = ties_before < ties_wanted ? min(e[u], ties_wanted - ties_before) : 0u;
        ties_before += e[u];
        mine += g[u] + allowed[u];
    }
    uint32_t out = kbeg + carry_sel + block_exclusive_scan(mine, warp_tot, sel_total);
    uint32_t tb = ties_before - esum;  // ties before this thread's first tile
#pragma unroll
    for (int u = 0; u < PER; ++u) {
        if (q0 + u < ntiles) {
            uint32_t *m = s.meta + ((int64_t)row * p.TT + first + q0 + u) * 4;
            s.outbase[(int64_t)row * (p.TT + 1) + first + q0 + u] = out;
            m[3] = allowed[u];
            m[2] = (tb + allowed[u] == ties_wanted && allowed[u] > 0) ? 1u : 0u;  // holds the last accepted tie
        }
        out += g[u] + allowed[u];
        tb += e[u];
    }
    // the last run sees the whole selection
    if (threadIdx.x == 0 && c0 + SCAN_PART >= ntiles && carry_sel + sel_total != k) atomicOr(p.status, STATUS_COUNT_MISMATCH);
}

// write: ordered compaction of a tile's candidate block into the message (one warp per tile)
__global__ void __launch_bounds__(THREADS) topk_write_kernel(const __grid_constant__ Params p, const TopkSide s) {
    const int row = blockIdx.y, lane = threadIdx.x & 31;
    const int tile = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (tile >= p.TT) return;
    const uint32_t out0 = s.outbase[(int64_t)row * (p.TT + 1) + tile];   // (fetched beside the segment lookup)
    const CandBlock cb = cand_block(p, s, tile, row);
    const uint32_t T = cb.sel[SEL_THRESH];
    const int64_t oend = (int64_t)row * p.K + __ldg(p.k_off + cb.t + 1);  // never write past the segment's slots
    if (cb.skip || cb.cnt == 0) return;
    const uint32_t allowed = cb.m.w;
    const bool has_last = cb.m.z != 0u;
    const int64_t obase = (int64_t)row * p.K + out0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t run_sel = 0, run_tie = 0;
    for (uint32_t c00 = 0; c00 < cb.cnt; c00 += 128) {   // four stripes of 32 candidates fetched before any is used
      float val4[4];
      uint32_t idx4[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
          const uint32_t q = c00 + 32 * u + lane;
          val4[u] = q < cb.cnt ? s.cand_val[cb.base + q] : 0.0f;
          idx4[u] = q < cb.cnt ? s.cand_idx[cb.base + q] : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t c0 = c00 + 32 * u;
        if (c0 >= cb.cnt) break;   // (uniform over the warp)
        const uint32_t q = c0 + lane;
        const bool in = q < cb.cnt;
        const float val = val4[u];
        const uint32_t idx = idx4[u];
        const uint32_t key = key_of(val);
        const bool tie = in && key == T;
        const uint32_t tb = __ballot_sync(0xffffffffu, tie);
        const uint32_t tie_rank = run_tie + __popc(tb & lt_mask);
        const bool take = in && (key > T || (tie && tie_rank < allowed));
        const uint32_t sb = __ballot_sync(0xffffffffu, take);
        if (take && obase + run_sel + __popc(sb & lt_mask) >= oend) {
            atomicOr(p.status, STATUS_COUNT_MISMATCH);  // inconsistent selection state: drop the write
        } else if (take) {
            const uint32_t out = run_sel + __popc(sb & lt_mask);
            s.idx[obase + out] = idx;
            s.val[obase + out] = val;
            if (s.zero_out) s.zero_out[idx] = 0.0f;
            if (has_last && tie && tie_rank == allowed - 1) cb.sel[SEL_CUT] = idx;
        }
        run_sel += __popc(sb);
        run_tie += __popc(tb);
      }
    }
}

// ------------------------------------------------------------------------------------------------
// Wide form, problems without candidates (SEL_FLAGS == 3: even the 24-bit prefix found by the dense
// second-digit pass leaves more entries than the buffer holds: huge groups of equal keys, e.g. a
// mostly-zero row whose k exceeds its non-zero count, or a vector of few distinct values).  Their
// tiles are walked in the dense source, tile-parallel: the last-digit histogram before pick 3, the
// per-tile counts before the scan, the ordered write after it; pick 3 and the scan treat them like
// any other problem.  Small strided grids that leave after one load when no problem needs them.
// ------------------------------------------------------------------------------------------------
template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_dense_hist3_kernel(const __grid_constant__ Params p, const TopkSide s) {
    __shared__ uint32_t h[DIGIT1_BINS];
    if (p.status[STATUS_ANY_DENSE + (s.zero_out ? 1 : 0)] == 0) return;
    const int row = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int tile = blockIdx.x; tile < p.TT; tile += gridDim.x) {
        const TileInfo ti = locate_tile(p, tile);
        uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        if (sel[SEL_FLAGS] != 3u || ti.seg_tiles == 1) continue;  // uniform over the CTA
        const uint32_t prefix = sel[SEL_PREFIX];
        for (int b = threadIdx.x; b < DIGIT1_BINS; b += THREADS) h[b] = 0u;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pos = tile_pos(warp, lane, j);
            float v[4];
            fetch4<GT>(s, row, ti, pos, v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t key = key_of(v[c]);
                if (pos + c < ti.len && (key >> 7) == prefix) atomicAdd(&h[key & 0x7fu], 1u);
            }
        }
        __syncthreads();
        flush_hist(h, s.hist2 + ((int64_t)row * p.T + ti.t) * DIGIT1_BINS, sel, SEL_LO2, SEL_HI2);
        __syncthreads();
    }
}

// entries above the threshold / equal to it per tile -> meta[2], meta[3] (what topk_count_kernel leaves)
template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_dense_count_kernel(const __grid_constant__ Params p, const TopkSide s) {
    __shared__ uint32_t wg[8], we[8];
    if (p.status[STATUS_ANY_DENSE + (s.zero_out ? 1 : 0)] == 0) return;
    const int row = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int tile = blockIdx.x; tile < p.TT; tile += gridDim.x) {
        const TileInfo ti = locate_tile(p, tile);
        const uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        if (sel[SEL_FLAGS] != 3u || ti.seg_tiles == 1) continue;  // uniform over the CTA
        const uint32_t T = sel[SEL_THRESH];
        uint32_t g = 0, e = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pos = tile_pos(warp, lane, j);
            float v[4];
            fetch4<GT>(s, row, ti, pos, v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t key = key_of(v[c]);
                const bool in = pos + c < ti.len;
                g += in && key > T ? 1u : 0u;
                e += in && key == T ? 1u : 0u;
            }
        }
        g = __reduce_add_sync(0xffffffffu, g);
        e = __reduce_add_sync(0xffffffffu, e);
        if (lane == 0) { wg[warp] = g; we[warp] = e; }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t *m = s.meta + ((int64_t)row * p.TT + tile) * 4;
            m[2] = wg[0] + wg[1] + wg[2] + wg[3] + wg[4] + wg[5] + wg[6] + wg[7];
            m[3] = we[0] + we[1] + we[2] + we[3] + we[4] + we[5] + we[6] + we[7];
        }
        __syncthreads();
    }
}

// ordered write of a dense tile's selected elements: one warp per tile, 32 consecutive elements per
// step (eight steps' elements fetched together); same rule as topk_write_kernel
template <typename GT>
__global__ void __launch_bounds__(THREADS) topk_dense_write_kernel(const __grid_constant__ Params p, const TopkSide s) {
    if (p.status[STATUS_ANY_DENSE + (s.zero_out ? 1 : 0)] == 0) return;
    const int row = blockIdx.y, lane = threadIdx.x & 31;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int tile = blockIdx.x * 8 + (threadIdx.x >> 5); tile < p.TT; tile += gridDim.x * 8) {
        const TileInfo ti = locate_tile(p, tile);
        uint32_t *sel = s.sel + ((int64_t)row * p.T + ti.t) * SEL_WORDS;
        if (sel[SEL_FLAGS] != 3u || ti.seg_tiles == 1) continue;  // uniform over the warp
        const uint32_t *m = s.meta + ((int64_t)row * p.TT + tile) * 4;
        const uint32_t T = sel[SEL_THRESH];
        const uint32_t allowed = m[3];
        const bool has_last = m[2] != 0u;
        const int64_t obase = (int64_t)row * p.K + s.outbase[(int64_t)row * (p.TT + 1) + tile];
        const int64_t oend = (int64_t)row * p.K + __ldg(p.k_off + ti.t + 1);  // never write past the segment's slots
        constexpr int SB = 8;
        uint32_t run_sel = 0, run_tie = 0;
        for (int c0 = 0; c0 < ti.len; c0 += 32 * SB) {
            float val[SB];
#pragma unroll
            for (int u = 0; u < SB; ++u)
                val[u] = c0 + 32 * u + lane < ti.len ? fetch1<GT>(s, row, ti.t, ti.seg_beg, ti.rel + c0 + 32 * u + lane) : 0.0f;
#pragma unroll
            for (int u = 0; u < SB; ++u) {
                if (c0 + 32 * u >= ti.len) break;   // (uniform over the warp)
                const int q = c0 + 32 * u + lane;
                const bool in = q < ti.len;
                const uint32_t idx = (uint32_t)(ti.seg_beg + ti.rel + q);
                const uint32_t key = key_of(val[u]);
                const bool tie = in && key == T;
                const uint32_t tb = __ballot_sync(0xffffffffu, tie);
                const uint32_t tie_rank = run_tie + __popc(tb & lt_mask);
                const bool take = in && (key > T || (tie && tie_rank < allowed));
                const uint32_t sb = __ballot_sync(0xffffffffu, take);
                if (take && obase + run_sel + __popc(sb & lt_mask) >= oend) {
                    atomicOr(p.status, STATUS_COUNT_MISMATCH);  // inconsistent selection state: drop the write
                } else if (take) {
                    const uint32_t out = run_sel + __popc(sb & lt_mask);
                    s.idx[obase + out] = idx;
                    s.val[obase + out] = val[u];
                    if (s.zero_out) s.zero_out[idx] = 0.0f;
                    if (has_last && tie && tie_rank == allowed - 1) sel[SEL_CUT] = idx;
                }
                run_sel += __popc(sb);
                run_tie += __popc(tb);
            }
        }
    }
}

// Wide form, last kernel of a side: closes the step's bookkeeping for every problem (one thread each).
__global__ void topk_close_kernel(const __grid_constant__ Params p, const TopkSide s) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x, row = blockIdx.y;
    if (t == 0 && row == 0) {
        if (s.spec) p.status[STATUS_ANY_REGULAR] = 0;   // the next step starts with "no problem on the regular route yet"
        p.status[STATUS_ANY_DENSE + (s.zero_out ? 1 : 0)] = 0;
    }
    if (t >= p.T) return;
    if (__ldg(p.tile_prefix + t + 1) - __ldg(p.tile_prefix + t) == 1) return;   // selected directly by one CTA
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    const uint32_t flags = sel[SEL_FLAGS];
    const bool single = s.spec && sel[SEL_MODE] == 1u;
    sel[SEL_CAND_COUNT] = 0u;
    sel[SEL_SPEC_FAIL] = 0u;
    sel[SEL_ROUTE] = (single ? ROUTE_SINGLE : 0) | ((flags & 2u) ? ROUTE_REFINED : 0) | ((flags & 1u) ? ROUTE_SLOW : 0);
}

// ------------------------------------------------------------------------------------------------
// Server pass for top-k uplink messages: one CTA per tile.
//   acc_j = sum over workers, in worker order, of the entries that hit j (absent entries add +0)
//   v_j   = e_j + acc_j / N   (written over e where it changes)
// fused with the first step of the downlink: first-digit histogram (top-k) or sign words and
// ||v||_1 partial (scaled sign).
// ------------------------------------------------------------------------------------------------
// TEL: also the tile's partial sums of e^2 (as read) and v^2 (as written), in tree order.
template <int DOWN, bool TEL>
__global__ void __launch_bounds__(THREADS, TEL ? 3 : 4) server_topk_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *acc = reinterpret_cast<float *>(smem_raw);                       // [TILE]
    uint32_t *h = reinterpret_cast<uint32_t *>(smem_raw + sizeof(float) * TILE);  // [DIGIT1_BINS] (top-k downlink)
    __shared__ double warp_sums[8];
    __shared__ double tel_sums[TEL ? 16 : 1];
    __shared__ uint32_t s_beg[16], s_end[16];  // this tile's range in each message of the current group of workers
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int q = threadIdx.x; q < TILE / 4; q += THREADS) reinterpret_cast<float4 *>(acc)[q] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    if (DOWN == COMP_TOPK)
        for (int b = threadIdx.x; b < DIGIT1_BINS / 4; b += THREADS) reinterpret_cast<uint4 *>(h)[b] = make_uint4(0u, 0u, 0u, 0u);
    // the tile of e is fetched now, so that its latency overlaps the message entries'
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0);
    float *e_tile = p.e + ti.seg_beg + ti.rel;
    float ev[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
        if (fast) load4_stream(e_tile + pos, ev[j]);
        else load4_guarded(e_tile, pos, ti.len, ev[j]);
    }
    double warp_e2 = 0.0;   // TEL: this warp's sum of e^2, kept while the messages are applied
    if constexpr (TEL) {
        double te[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) te[j] = leaf4_sq(ev[j]);
        warp_e2 = warp_tree_reduce8(te, lane);
    }
    __syncthreads();
    const bool last_tile = (blockIdx.x + 1 == __ldg(p.tile_prefix + ti.t + 1));
    const uint32_t tile_first = (uint32_t)(ti.seg_beg + ti.rel);
    // Workers are taken 8 at a time.  Thread q first fetches entry q of this tile from each of the
    // 8 messages (all fetches in flight together); then the entries are added worker by worker, one
    // barrier apart, so that every element sees its contributions in worker order.  Inside one
    // worker's turn the indices are distinct, so its additions do not depend on one another.
    constexpr int WG = 8;
    const int tid = threadIdx.x, num_workers = p.N;
    const int64_t K = p.K;
    const uint32_t *idx_row = p.up_idx;   // the current group's first message
    const float *val_row = p.up_val;
    for (int g0 = 0; g0 < num_workers; g0 += WG, idx_row += WG * K, val_row += WG * K) {
        if (tid < WG) {
            const int i = g0 + tid;
            uint32_t beg = 0, end = 0;
            if (i < num_workers) {
                const uint32_t *ob = p.up_outbase + (int64_t)i * (p.TT + 1) + blockIdx.x;
                beg = ob[0];
                end = last_tile ? (uint32_t)__ldg(p.k_off + ti.t + 1) : ob[1];
            }
            s_beg[tid] = beg;
            s_end[tid] = end;
        }
        __syncthreads();
        uint32_t pidx[WG];
        float pval[WG];
        uint32_t crowded = 0;   // workers with more than 256 entries in this tile (uniform over the CTA)
        {
            const uint32_t *ip = idx_row;
            const float *vp = val_row;
#pragma unroll
            for (int u = 0; u < WG; ++u, ip += K, vp += K) {
                const uint32_t q = s_beg[u] + tid;
                const bool have = q < s_end[u];   // (beg = end = 0 for workers beyond N)
                crowded |= (s_end[u] - s_beg[u] > (uint32_t)THREADS ? 1u : 0u) << u;
                pidx[u] = have ? ip[q] : 0xffffffffu;
                pval[u] = have ? vp[q] : 0.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < WG; ++u) {
            if (g0 + u < num_workers) {  // uniform over the CTA
                const uint32_t o = pidx[u] - tile_first;
                if (o < (uint32_t)TILE) acc[o] = __fadd_rn(acc[o], pval[u]);  // (absent entries and those of a refused subset fall outside)
                if ((crowded >> u) & 1u) {
                    const uint32_t *idx = idx_row + (int64_t)u * K;
                    const float *val = val_row + (int64_t)u * K;
                    for (uint32_t q = s_beg[u] + tid + THREADS; q < s_end[u]; q += THREADS) {
                        const uint32_t o2 = idx[q] - tile_first;
                        if (o2 < (uint32_t)TILE) acc[o2] = __fadd_rn(acc[o2], val[q]);
                    }
                }
                __syncthreads();
            }
        }
    }
    const WorkerDivisor by_n(p.N);
    const bool with_hist = ti.seg_tiles > 1;   // (single-tile segments are selected directly from v)
    const int64_t wbase = __ldg(p.word_off + ti.t) + ti.rel / 32;
    const int nwords = (ti.len + 31) >> 5;
    double a[8];
    double tv[TEL ? 8 : 1];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
        float v[4];
        const float4 a4 = *reinterpret_cast<const float4 *>(&acc[pos]);
        const float av[4] = {a4.x, a4.y, a4.z, a4.w};
        by_n.div4(av, v);
        if (fast) {   // one 128-bit store when any of the four changed (the others are rewritten with their own bits)
            bool changed = false;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                v[c] = __fadd_rn(ev[j][c], v[c]);
                changed |= __float_as_uint(v[c]) != __float_as_uint(ev[j][c]);
                if (DOWN == COMP_TOPK && with_hist) atomicAdd(&h[key_of(v[c]) >> DIGIT1_SHIFT], 1u);
            }
            if (changed) *reinterpret_cast<float4 *>(e_tile + pos) = make_float4(v[0], v[1], v[2], v[3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const bool valid = pos + c < ti.len;
                v[c] = __fadd_rn(ev[j][c], v[c]);
                if (!valid) v[c] = 0.0f;
                if (valid && __float_as_uint(v[c]) != __float_as_uint(ev[j][c])) e_tile[pos + c] = v[c];
                if (DOWN == COMP_TOPK && valid && with_hist) atomicAdd(&h[key_of(v[c]) >> DIGIT1_SHIFT], 1u);
            }
        }
        if constexpr (TEL) tv[j] = leaf4_sq(v);
        if (DOWN == COMP_SIGN) {
            a[j] = leaf4(v);
            uint32_t w = pack_word(sign_nibble(v), lane);
            int widx = warp * 32 + j * 4 + (lane >> 3);
            if ((lane & 7) == 0 && widx < nwords) p.down_words[wbase + widx] = w;
        }
    }
    if (DOWN == COMP_SIGN) {
        double sum = cta_tree_reduce(warp_tree_reduce8(a, lane), warp_sums);
        if (threadIdx.x == 0) p.down_partials[blockIdx.x] = sum;
    }
    if constexpr (TEL) {
        double re, rv;
        cta_tree_reduce_pair(warp_e2, warp_tree_reduce8(tv, lane), tel_sums, re, rv);
        if (threadIdx.x == 0) { p.tel_e[blockIdx.x] = re; p.tel_v[blockIdx.x] = rv; }
    }
    if (DOWN == COMP_TOPK && ti.seg_tiles > 1) {   // (single-tile segments are selected directly from v)
        __syncthreads();
        flush_hist(h, p.down_hist + (int64_t)ti.t * DIGIT1_BINS, p.down_sel + (int64_t)ti.t * SEL_WORDS, SEL_LO1, SEL_HI1);
    }
}

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
#define CHECK_LAUNCH()                                   \
    do {                                                 \
        cudaError_t e__ = cudaGetLastError();            \
        if (e__ != cudaSuccess) return e__;              \
        ++*launches;                                     \
    } while (0)

// Grid of the dense passes that usually have nothing to do on the uplink (their CTAs walk the
// tiles with a stride and leave at once when no problem takes the regular route).
static dim3 strided_grid(const Params &p, int rows) {
    const int per_row = (2368 + rows - 1) / rows;  // about 16 CTAs per SM over all rows
    return dim3(p.TT < per_row ? p.TT : per_row, rows);
}

// Candidate histograms of the wide form.  Segments below LONG_SEG_TILES tiles: a warp per tile block,
// 16 tiles per CTA (many warps in flight on what is a chain of dependent loads per block).  Longer
// segments: their candidate regions as a whole, 8192 or 32768 candidates per CTA.
static cudaError_t launch_cand_hist(const Params &p, const TopkSide &s, int level, cudaStream_t st, int64_t *launches) {
    if (p.n_long < p.n_large) {
        constexpr int REPS = 2;
        topk_cand_hist_kernel<<<dim3((p.TT + 8 * REPS - 1) / (8 * REPS), s.R), THREADS, 0, st>>>(p, s, level, REPS);
        CHECK_LAUNCH();
    }
    if (p.n_long > 0) {
        // (four runs per CTA from 2^24 candidate slots up; three more positions cover a region that starts off a 16-byte boundary)
        const int batches = s.cap_long_max * p.n_long * s.R >= (int64_t)1 << 24 ? 4 : 1;
        const int64_t per_cta = (int64_t)batches * CAND_RUN;
        const int chunks = (int)((s.cap_long_max + 3 + per_cta - 1) / per_cta);
        topk_cand_hist_long_kernel<<<dim3(p.n_long * chunks, s.R), THREADS, 0, st>>>(p, s, level, chunks, batches);
        CHECK_LAUNCH();
    }
    return cudaSuccess;
}

// First part of a side (multi-tile segments).  Uplink: candidates are
// collected with last step's guess and the guess is checked; then, for the problems left on the
// regular route, the first-digit histogram.  Downlink without a fused histogram: plain first-digit
// histogram of v.
// One launch of a kernel template over the element type of the side's source.
#define LAUNCH_BY_SOURCE(kernel, grid, ...)                                                      \
    do {                                                                                         \
        if (src_kind == SRC_BF16) kernel<__nv_bfloat16 __VA_ARGS__><<<grid, THREADS, 0, st>>>(p, s); \
        else if (src_kind == SRC_SCORES) kernel<ScoreGen __VA_ARGS__><<<grid, THREADS, 0, st>>>(p, s);  \
        else kernel<float __VA_ARGS__><<<grid, THREADS, 0, st>>>(p, s);                           \
        CHECK_LAUNCH();                                                                          \
    } while (0)
#define COMMA ,

cudaError_t topk_first_part(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st, int64_t *launches) {
    dim3 g_tiles(p.TT, s.R), g_probs(p.T, s.R);
    if (!p.n_large) return cudaSuccess;
    if (s.spec) {
        LAUNCH_BY_SOURCE(topk_filter_tma_kernel, g_tiles, COMMA true);
        cudaError_t e = launch_topk_check(p, s, st);
        if (e != cudaSuccess) return e;
        ++*launches;
        if (!use_fused_tail(p)) {   // wide form: first digit of the single-pass problems from a global histogram
            if ((e = launch_cand_hist(p, s, 0, st, launches)) != cudaSuccess) return e;
            topk_pick_kernel<<<g_probs, THREADS, 0, st>>>(p, s, 5); CHECK_LAUNCH();
        }
    }
    const dim3 g_hist = s.spec ? strided_grid(p, s.R) : g_tiles;
    LAUNCH_BY_SOURCE(topk_hist1_kernel, g_hist);
    return cudaSuccess;
}

cudaError_t launch_topk_hist1(const Params &p, bool uplink, cudaStream_t st, int64_t *launches) {
    return topk_first_part(p, make_side(p, uplink), uplink && p.gdt == DT_BF16 ? SRC_BF16 : SRC_F32, st, launches);
}

// Everything after the first-digit histogram: the message, the thresholds, and for the
// downlink the zeroing of the selected error entries.
cudaError_t topk_second_part(const Params &p, const TopkSide &s, int src_kind, cudaStream_t st, int64_t *launches) {
    dim3 g_tiles(p.TT, s.R), g_probs(p.T, s.R), g_warp_tiles((p.TT + 7) / 8, s.R);
    if (!p.n_large) return cudaSuccess;
    topk_pick_kernel<<<g_probs, THREADS, 0, st>>>(p, s, 1); CHECK_LAUNCH();
    const dim3 g_strided = strided_grid(p, s.R);
    LAUNCH_BY_SOURCE(topk_hist2_dense_kernel, g_strided);
    topk_pick_kernel<<<g_probs, THREADS, 0, st>>>(p, s, 4); CHECK_LAUNCH();
    const dim3 g_filter = s.spec ? strided_grid(p, s.R) : g_tiles;
    LAUNCH_BY_SOURCE(topk_filter_tma_kernel, g_filter, COMMA false);
    if (use_fused_tail(p)) return launch_topk_tail(p, s, src_kind, st, launches);
    // some segment has too many candidates or tiles for one CTA: the same steps, spread over the tile blocks
    cudaError_t e;
    if ((e = launch_cand_hist(p, s, 1, st, launches)) != cudaSuccess) return e;
    topk_pick_kernel<<<g_probs, THREADS, 0, st>>>(p, s, 2); CHECK_LAUNCH();
    if ((e = launch_cand_hist(p, s, 2, st, launches)) != cudaSuccess) return e;
    LAUNCH_BY_SOURCE(topk_dense_hist3_kernel, g_strided);
    topk_pick_kernel<<<g_probs, THREADS, 0, st>>>(p, s, 3); CHECK_LAUNCH();
    topk_count_kernel<<<g_warp_tiles, THREADS, 0, st>>>(p, s); CHECK_LAUNCH();
    LAUNCH_BY_SOURCE(topk_dense_count_kernel, g_strided);
    const dim3 g_scan(p.T * p.scan_parts, s.R);
    if (p.scan_parts > 1) { topk_scan_kernel<<<g_scan, THREADS, 0, st>>>(p, s, 0); CHECK_LAUNCH(); }
    topk_scan_kernel<<<g_scan, THREADS, 0, st>>>(p, s, 1); CHECK_LAUNCH();
    topk_write_kernel<<<g_warp_tiles, THREADS, 0, st>>>(p, s); CHECK_LAUNCH();
    LAUNCH_BY_SOURCE(topk_dense_write_kernel, g_strided);
    topk_close_kernel<<<dim3((p.T + 127) / 128, s.R), 128, 0, st>>>(p, s); CHECK_LAUNCH();
    return cudaSuccess;
}

cudaError_t launch_topk_select(const Params &p, bool uplink, cudaStream_t st, int64_t *launches) {
    return topk_second_part(p, make_side(p, uplink), uplink && p.gdt == DT_BF16 ? SRC_BF16 : SRC_F32, st, launches);
}

constexpr size_t SERVER_TOPK_SMEM = sizeof(float) * TILE + sizeof(uint32_t) * DIGIT1_BINS;

cudaError_t configure_topk_kernels() {
    cudaError_t e = configure_topk_tail_kernels();
    const void *kernels[] = {(const void *)server_topk_kernel<COMP_TOPK, false>, (const void *)server_topk_kernel<COMP_SIGN, false>,
                             (const void *)server_topk_kernel<COMP_IDENTITY, false>, (const void *)server_topk_kernel<COMP_TOPK, true>,
                             (const void *)server_topk_kernel<COMP_SIGN, true>, (const void *)server_topk_kernel<COMP_IDENTITY, true>};
    for (const void *k : kernels)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SERVER_TOPK_SMEM);
    return e;
}

// Single-tile segments of one side, selected directly (independent of everything else on that side:
// the caller may run it on a stream of its own).
cudaError_t launch_topk_small_segments(const Params &p, bool uplink, cudaStream_t st, int64_t *launches) {
    if (!p.n_small) return cudaSuccess;
    const TopkSide s = make_side(p, uplink);
    cudaError_t e = launch_topk_small(p, s, uplink && p.gdt == DT_BF16 ? SRC_BF16 : SRC_F32, st);
    if (e == cudaSuccess) ++*launches;
    return e;
}

// ------------------------------------------------------------------------------------------------
// Seeded draw of the random-k subsets (Def. 3): every element of a segment gets a pseudo-random
// 30-bit score (philox.cuh) and the k_t highest scores are the segment's subset, equal scores to the
// lower index.  That is a top-k selection on a vector that is computed instead of read, so the
// kernels above run it unchanged, with ScoreGen as their source type: rows 0..N-1 are the workers'
// subsets, row N the server's; the output "message" is the subset list itself (ascending indices).
// Scores are uniform, so the threshold is known in advance up to sampling noise: the single-pass
// route starts from that bound instead of last step's threshold (and, like every guess, is checked).
// ------------------------------------------------------------------------------------------------
__global__ void randk_draw_begin_kernel(const __grid_constant__ Params p, const TopkSide s) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x, row = blockIdx.y;
    if (t >= p.T) return;
    if (__ldg(p.tile_prefix + t + 1) - __ldg(p.tile_prefix + t) == 1) return;   // selected directly
    uint32_t *sel = s.sel + ((int64_t)row * p.T + t) * SEL_WORDS;
    const double n = (double)(__ldg(p.seg_off + t + 1) - __ldg(p.seg_off + t));
    const double k = (double)(__ldg(p.k_off + t + 1) - __ldg(p.k_off + t));
    // candidates wanted: k plus six standard deviations of their count and some more
    const double want = k + 6.0 * sqrt(k) + 64.0;
    uint32_t bound = 1u;   // (0 would mean "no guess")
    if (want < n) bound = max(1u, (uint32_t)(1073741824.0 * (1.0 - want / n)));
    sel[SEL_GUESS] = bound;
}

// The single-tile segments of the draw (independent of the rest: the caller may put them on a stream of their own).
cudaError_t launch_randk_draw_small(const Params &p, const TopkSide &s, cudaStream_t st, int64_t *launches) {
    if (!p.n_small) return cudaSuccess;
    cudaError_t e = launch_topk_small(p, s, SRC_SCORES, st);
    if (e == cudaSuccess) ++*launches;
    return e;
}

// The multi-tile segments of the draw.
cudaError_t launch_randk_draw(const Params &p, const TopkSide &s, cudaStream_t st, int64_t *launches) {
    if (!p.n_large) return cudaSuccess;
    randk_draw_begin_kernel<<<dim3((p.T + 127) / 128, s.R), 128, 0, st>>>(p, s);
    CHECK_LAUNCH();
    cudaError_t e = topk_first_part(p, s, SRC_SCORES, st, launches);
    if (e != cudaSuccess) return e;
    return topk_second_part(p, s, SRC_SCORES, st, launches);
}

template <bool TEL>
static void launch_server_topk_t(const Params &p, cudaStream_t st) {
    if (p.down == COMP_TOPK) server_topk_kernel<COMP_TOPK, TEL><<<p.TT, THREADS, SERVER_TOPK_SMEM, st>>>(p);
    else if (p.down == COMP_SIGN) server_topk_kernel<COMP_SIGN, TEL><<<p.TT, THREADS, SERVER_TOPK_SMEM, st>>>(p);
    else server_topk_kernel<COMP_IDENTITY, TEL><<<p.TT, THREADS, SERVER_TOPK_SMEM, st>>>(p);
}

cudaError_t launch_server_topk(const Params &p, cudaStream_t st, int64_t *launches) {
    if (p.telemetry) launch_server_topk_t<true>(p, st);
    else launch_server_topk_t<false>(p, st);
    CHECK_LAUNCH();
    return cudaSuccess;
}

}  // namespace liec
