// Device helpers shared by the tile kernels: tile lookup, 4-wide loads, the balanced
// binary64 tree over a warp's 1024 elements, sign-word packing.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "plan.h"

namespace liec {

struct TileInfo {
    int t;            // segment
    int64_t seg_beg;  // first element of the segment within a row
    int64_t n;        // segment length
    int64_t rel;      // first element of the tile, relative to the segment
    int len;          // valid elements in the tile (1..TILE)
    int tile_in_seg;  // tile index inside the segment
    int seg_tiles;    // tiles of the segment
};

// Segment and extent of tile `tile` (table lookups only).
__device__ __forceinline__ TileInfo locate_tile(const Params &p, int tile) {
    TileInfo ti;
    ti.t = __ldg(p.tile_seg + tile);
    ti.seg_beg = __ldg(p.seg_off + ti.t);
    ti.n = __ldg(p.seg_off + ti.t + 1) - ti.seg_beg;
    const int first_tile = __ldg(p.tile_prefix + ti.t);
    ti.tile_in_seg = tile - first_tile;
    ti.seg_tiles = __ldg(p.tile_prefix + ti.t + 1) - first_tile;
    ti.rel = (int64_t)ti.tile_in_seg * TILE;
    int64_t left = ti.n - ti.rel;
    ti.len = left < TILE ? (int)left : TILE;
    return ti;
}

// ---- 4 consecutive gradient elements, widened to binary32 --------------------------------

__device__ __forceinline__ void load4_stream(const float *ptr, float (&v)[4]) {
    float4 q = __ldcs(reinterpret_cast<const float4 *>(ptr));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4_stream(const __nv_bfloat16 *ptr, float (&v)[4]) {
    uint2 q = __ldcs(reinterpret_cast<const uint2 *>(ptr));
    v[0] = __uint_as_float(q.x << 16);
    v[1] = __uint_as_float(q.x & 0xffff0000u);
    v[2] = __uint_as_float(q.y << 16);
    v[3] = __uint_as_float(q.y & 0xffff0000u);
}
// Same, through the normal caching path (for data that is read again soon).
__device__ __forceinline__ void load4_cached(const float *ptr, float (&v)[4]) {
    float4 q = __ldg(reinterpret_cast<const float4 *>(ptr));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4_cached(const __nv_bfloat16 *ptr, float (&v)[4]) {
    uint2 q = __ldg(reinterpret_cast<const uint2 *>(ptr));
    v[0] = __uint_as_float(q.x << 16);
    v[1] = __uint_as_float(q.x & 0xffff0000u);
    v[2] = __uint_as_float(q.y << 16);
    v[3] = __uint_as_float(q.y & 0xffff0000u);
}
__device__ __forceinline__ float load1(const float *ptr) { return *ptr; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *ptr) {
    return __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(ptr)) << 16);
}
// Guarded scalar version: elements at or beyond `len` read as +0.
template <typename GT>
__device__ __forceinline__ void load4_guarded(const GT *tile_ptr, int pos, int len, float (&v)[4]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = (pos + c < len) ? load1(tile_ptr + pos + c) : 0.0f;
}

// Copies a ragged or misaligned tile into shared memory with ordinary loads; positions at or beyond
// `len` become +0.  With a 16-byte aligned source whole 16-byte chunks move at once (the chunk
// that straddles `len` is assembled element by element by the thread that owns it); several loads
// per thread are in flight either way.  The caller synchronises afterwards.
template <typename T>
__device__ __forceinline__ void stage_tile_guarded(T *dst, const T *src, int len, bool aligned16) {
    constexpr int PER = 16 / (int)sizeof(T);
    if (aligned16) {
        const int full = len / PER;
#pragma unroll 4
        for (int c = threadIdx.x; c < TILE / PER; c += THREADS) {
            if (c < full) {
                reinterpret_cast<uint4 *>(dst)[c] = __ldcs(reinterpret_cast<const uint4 *>(src) + c);
            } else if (c > full) {
                reinterpret_cast<uint4 *>(dst)[c] = make_uint4(0u, 0u, 0u, 0u);
            } else {
#pragma unroll
                for (int e = 0; e < PER; ++e) dst[c * PER + e] = (c * PER + e < len) ? src[c * PER + e] : T(0);
            }
        }
    } else {
#pragma unroll 8
        for (int q = threadIdx.x; q < TILE; q += THREADS) dst[q] = q < len ? src[q] : T(0);
    }
}

// a / N in binary32, round to nearest even.  When N is a power of two, a / N and a * (1/N) are the
// same real number (1/N is exact), so one multiplication rounds to the same float as the IEEE
// division, subnormal results included; every other N takes the division.
struct WorkerDivisor {
    float n, inv;
    bool pow2;
    __device__ __forceinline__ explicit WorkerDivisor(int N) : n((float)N), inv(1.0f / (float)N), pow2((N & (N - 1)) == 0) {}
    __device__ __forceinline__ float operator()(float a) const { return pow2 ? __fmul_rn(a, inv) : __fdiv_rn(a, n); }
    __device__ __forceinline__ void div4(const float (&a)[4], float (&q)[4]) const {
        if (pow2) {
#pragma unroll
            for (int c = 0; c < 4; ++c) q[c] = __fmul_rn(a[c], inv);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) q[c] = __fdiv_rn(a[c], n);
        }
    }
};

// Position (relative to the tile) of the 4 elements a thread owns in row j of its warp.
__device__ __forceinline__ int tile_pos(int warp, int lane, int j) { return warp * 1024 + j * 128 + lane * 4; }

// ---- balanced binary64 tree -----------------------------------------------------------------
//
// A warp owns 1024 consecutive elements as 8 rows of 128; lane l of row j owns elements
// 4l..4l+3 of that row.  leaf4 sums a lane's 4 magnitudes (two tree levels).  The warp
// reduction then follows the tree upwards: lanes xor 1,2,4,8,16 inside each row, then rows
// pairwise.  Rows are folded across lanes while reducing ("transposed" butterfly) so that
// each level costs one shuffle+add per surviving value instead of one per row.

__device__ __forceinline__ double leaf4(const float (&v)[4]) {
    double a0 = (double)fabsf(v[0]), a1 = (double)fabsf(v[1]);
    double a2 = (double)fabsf(v[2]), a3 = (double)fabsf(v[3]);
    return __dadd_rn(__dadd_rn(a0, a1), __dadd_rn(a2, a3));
}

// Same two levels over the squares (telemetry: squared norms over the same tree).  A binary32
// value squared is exact in binary64 (24-bit significands).
__device__ __forceinline__ double leaf4_sq(const float (&v)[4]) {
    const double d0 = (double)v[0], d1 = (double)v[1], d2 = (double)v[2], d3 = (double)v[3];
    return __dadd_rn(__dadd_rn(__dmul_rn(d0, d0), __dmul_rn(d1, d1)), __dadd_rn(__dmul_rn(d2, d2), __dmul_rn(d3, d3)));
}

__device__ __forceinline__ double shfl_xor_f64(double x, int mask) {
    return __shfl_xor_sync(0xffffffffu, x, mask);
}

// a[j] = this lane's leaf sum in row j (ROWS rows per warp, ROWS = 8 or 4).  Returns, in every
// lane, the tree sum of the warp's 1024 elements.
template <int ROWS>
__device__ __forceinline__ double warp_tree_reduce(double (&a)[ROWS], int lane) {
    constexpr int LOG = ROWS == 8 ? 3 : 2;
    // lane levels 1,2,(4) while folding ROWS rows -> 1 value per lane
#pragma unroll
    for (int step = 0; step < LOG; ++step) {
        const int m = 1 << step;
        const int half = (ROWS / 2) >> step;
        const bool upper = (lane & m) != 0;
#pragma unroll
        for (int r = 0; r < half; ++r) {
            double send = upper ? a[r] : a[r + half];
            double keep = upper ? a[r + half] : a[r];
            double recv = shfl_xor_f64(send, m);
            a[r] = __dadd_rn(keep, recv);
        }
    }
    double s = a[0];
    // remaining lane levels of the row this lane now represents
#pragma unroll
    for (int m = ROWS; m < 32; m <<= 1) s = __dadd_rn(s, shfl_xor_f64(s, m));
    // row levels: row bit b lives in lane bit LOG-1-b
#pragma unroll
    for (int m = ROWS / 2; m >= 1; m >>= 1) s = __dadd_rn(s, shfl_xor_f64(s, m));
    return s;
}

__device__ __forceinline__ double warp_tree_reduce8(double (&a)[8], int lane) { return warp_tree_reduce<8>(a, lane); }

// Combine the 8 warp sums of a CTA (tile of 8192 elements) in tree order; result in thread 0.
__device__ __forceinline__ double cta_tree_reduce(double warp_sum, double *smem8) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem8[warp] = warp_sum;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0) {
        double s01 = __dadd_rn(smem8[0], smem8[1]), s23 = __dadd_rn(smem8[2], smem8[3]);
        double s45 = __dadd_rn(smem8[4], smem8[5]), s67 = __dadd_rn(smem8[6], smem8[7]);
        s = __dadd_rn(__dadd_rn(s01, s23), __dadd_rn(s45, s67));
    }
    return s;
}

// Two tile sums at once (one barrier): results in thread 0.
__device__ __forceinline__ void cta_tree_reduce_pair(double wa, double wb, double *smem16, double &ra, double &rb) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { smem16[warp] = wa; smem16[8 + warp] = wb; }
    __syncthreads();
    ra = rb = 0.0;
    if (threadIdx.x == 0) {
        const double *a = smem16, *b = smem16 + 8;
        ra = __dadd_rn(__dadd_rn(__dadd_rn(a[0], a[1]), __dadd_rn(a[2], a[3])), __dadd_rn(__dadd_rn(a[4], a[5]), __dadd_rn(a[6], a[7])));
        rb = __dadd_rn(__dadd_rn(__dadd_rn(b[0], b[1]), __dadd_rn(b[2], b[3])), __dadd_rn(__dadd_rn(b[4], b[5]), __dadd_rn(b[6], b[7])));
    }
}

// Combines per-tile partial sums (binary64) of one segment in tree order: pairwise, level by level,
// over the tile count zero-padded to a power of two (adding +0 is exact), which continues the
// segment's balanced tree above the tile level.  Segments of more than FIN_CHUNK tiles are reduced
// chunk by chunk (a chunk of FIN_CHUNK tiles is an aligned subtree) and the chunk sums are combined
// by the same rule.  Whole CTA (THREADS threads); the result is valid in thread 0.
constexpr int FIN_CHUNK = 2048;
constexpr int FIN_MAX_CHUNKS = 256;  // 2^32 elements / TILE / FIN_CHUNK

__device__ __forceinline__ double tree_reduce_partials(const double *src, int ntiles, double *buf /*[FIN_CHUNK]*/,
                                                       double *chunk_sums /*[FIN_MAX_CHUNKS]*/) {
    const int nchunks = (ntiles + FIN_CHUNK - 1) / FIN_CHUNK;
    for (int c = 0; c < nchunks; ++c) {
        // the chunk's tree over the next power of two of its tile count: the levels above it would
        // only add +0, which changes nothing
        const int here = min(FIN_CHUNK, ntiles - c * FIN_CHUNK);
        int span = 1;
        while (span < here) span <<= 1;
        for (int q = threadIdx.x; q < span; q += THREADS) {
            const int idx = c * FIN_CHUNK + q;
            buf[q] = idx < ntiles ? src[idx] : 0.0;
        }
        __syncthreads();
        for (int width = span / 2; width >= 1; width >>= 1) {
            // pairwise: new[q] = old[2q] + old[2q+1]; done in two phases to avoid overwrite hazards
            double vals[FIN_CHUNK / 2 / THREADS];
#pragma unroll
            for (int r = 0; r < FIN_CHUNK / 2 / THREADS; ++r) {
                const int q = threadIdx.x + r * THREADS;
                vals[r] = q < width ? __dadd_rn(buf[2 * q], buf[2 * q + 1]) : 0.0;
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < FIN_CHUNK / 2 / THREADS; ++r) {
                const int q = threadIdx.x + r * THREADS;
                if (q < width) buf[q] = vals[r];
            }
            __syncthreads();
        }
        if (threadIdx.x == 0) chunk_sums[c] = buf[0];
        __syncthreads();
    }
    double total = 0.0;
    if (threadIdx.x == 0) {
        int L = 1;
        while (L < nchunks) L <<= 1;
        for (int c = nchunks; c < L; ++c) chunk_sums[c] = 0.0;
        for (int width = L / 2; width >= 1; width >>= 1)
            for (int q = 0; q < width; ++q) chunk_sums[q] = __dadd_rn(chunk_sums[2 * q], chunk_sums[2 * q + 1]);
        total = chunk_sums[0];
    }
    return total;
}

// ---- sign words -------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t sign_nibble(const float (&v)[4]) {
    return (v[0] < 0.0f ? 1u : 0u) | (v[1] < 0.0f ? 2u : 0u) | (v[2] < 0.0f ? 4u : 0u) | (v[3] < 0.0f ? 8u : 0u);
}

// The 8 lanes that share a 32-element word OR their nibbles together; every lane of the
// group gets the word.
__device__ __forceinline__ uint32_t pack_word(uint32_t nibble, int lane) {
    uint32_t w = nibble << (4 * (lane & 7));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    return w;
}

// Scaled sign of one tile held in global memory (4-wide layout): writes the tile's sign words and
// returns, in thread 0, the binary64 tree sum of its magnitudes.  `fast`: the tile is full and its
// first element 16-byte aligned.  Whole CTA.
template <typename GT>
__device__ __forceinline__ double sign_tile(const GT *tile_ptr, int len, bool fast, uint32_t *tile_words,
                                            double *warp_sums /*[8]*/) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float v[8][4];
    if (fast) {
#pragma unroll
        for (int j = 0; j < 8; ++j) load4_stream(tile_ptr + tile_pos(warp, lane, j), v[j]);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) load4_guarded(tile_ptr, tile_pos(warp, lane, j), len, v[j]);
    }
    const int nwords = (len + 31) >> 5;
    double a[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        a[j] = leaf4(v[j]);
        const uint32_t w = pack_word(sign_nibble(v[j]), lane);
        const int widx = warp * 32 + j * 4 + (lane >> 3);
        if ((lane & 7) == 0 && widx < nwords) tile_words[widx] = w;
    }
    return cta_tree_reduce(warp_tree_reduce8(a, lane), warp_sums);
}

// Nibble of this lane's 4 elements in row j, taken from the warp's 32 words (lane l holds word l).
__device__ __forceinline__ uint32_t nibble_from_words(uint32_t my_word, int lane, int j) {
    uint32_t w = __shfl_sync(0xffffffffu, my_word, 4 * j + (lane >> 3));
    return (w >> (4 * (lane & 7))) & 0xfu;
}

// ---- bulk copies into shared memory (TMA, untiled) and their bounded waits -----------------------

__device__ __forceinline__ uint32_t smem_u32(const void *ptr) { return (uint32_t)__cvta_generic_to_shared(ptr); }

// One thread: announce `expect` bytes on the mbarrier and start a bulk copy of `bytes` bytes
// (both addresses 16-byte aligned, bytes a multiple of 16).  expect == bytes in normal operation.
__device__ __forceinline__ void bulk_copy_g2s(void *dst_smem, const void *src, uint32_t bytes, uint32_t expect,
                                              unsigned long long *bar) {
    const uint32_t b = smem_u32(bar);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // earlier generic accesses of the buffer come first
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(expect) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(b) : "memory");
}

// Polls the mbarrier's phase `parity` at most `limit` times; true when the phase completed.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, uint32_t parity, uint32_t limit) {
    uint32_t done = 0;
    const uint32_t b = smem_u32(bar);
    for (uint32_t spin = 0; spin < limit && !done; ++spin)
        asm volatile("{ .reg .pred q; mbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2; selp.u32 %0, 1, 0, q; }"
                     : "=r"(done) : "r"(b), "r"(parity) : "memory");
    return done != 0;
}

// After a wait that ran out: before the CTA gives its shared memory back, give a copy that may
// still be in flight time to land.  Polls until the phase completes, but for at least a
// millisecond (a healthy copy of a tile takes microseconds) and at most 2^22 polls.
__device__ __forceinline__ bool mbar_drain(unsigned long long *bar, uint32_t parity) {
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (uint32_t round = 0; round < (1u << 12); ++round) {
        if (mbar_wait_bounded(bar, parity, 1u << 10)) return true;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > 1000000ull) break;
    }
    return false;
}

}  // namespace liec
