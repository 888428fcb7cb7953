// Model-averaging iteration of Algorithm 1 (the branch taken every floor(1/delta)-th step; the
// experiments fix the period at 32 or 100) and the algorithm's output, the mean model.
//
//   v = e + (1/N) sum_i g^i,  p = v,  e <- v - p = +0,
//   xbar = (1/N) sum_i x^i,   x^i <- xbar - eta ((p - g^i) + g^i)
//
// One CTA per tile does the whole iteration for its 8192 coordinates: a first sweep over the
// workers accumulates the gradient and model sums in worker order, a second sweep re-reads each
// worker's gradients (from L2: a tile's N rows are N x 16-32 KB) and writes the new models.
#include "device_common.cuh"
#include "kernels.h"

namespace liec {

// FAST: every worker's row of this tile is full and 16-byte aligned (the same for all workers, so
// the sweeps over the workers carry no branch and their loads can be issued several workers ahead).
template <typename GT, bool FAST>
__device__ __forceinline__ void average_tile(const Params &p, const TileInfo &ti, const float lr, const int j0) {
    constexpr int HR = 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float gs[HR][4], xs[HR][4];
#pragma unroll
    for (int j = 0; j < HR; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) { gs[j][c] = 0.0f; xs[j][c] = 0.0f; }
    const GT *g_tile0 = reinterpret_cast<const GT *>(p.G) + ti.seg_beg + ti.rel;
    float *x_tile0 = p.X + ti.seg_beg + ti.rel;
#pragma unroll 2
    for (int i = 0; i < p.N; ++i) {
        const GT *g_tile = g_tile0 + (int64_t)i * p.d;
        const float *x_tile = x_tile0 + (int64_t)i * p.d;
#pragma unroll
        for (int j = 0; j < HR; ++j) {
            const int pos = tile_pos(warp, lane, j0 + j);
            float g[4], x[4];
            if (FAST) { load4_cached(g_tile + pos, g); load4_stream(x_tile + pos, x); }
            else { load4_guarded(g_tile, pos, ti.len, g); load4_guarded(x_tile, pos, ti.len, x); }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                gs[j][c] = __fadd_rn(gs[j][c], g[c]);
                xs[j][c] = __fadd_rn(xs[j][c], x[c]);
            }
        }
    }
    const WorkerDivisor by_n(p.N);
    float *e_tile = p.e + ti.seg_beg + ti.rel;
#pragma unroll
    for (int j = 0; j < HR; ++j) {
        const int pos = tile_pos(warp, lane, j0 + j);
        float ev[4];
        if (FAST) load4_stream(e_tile + pos, ev);
        else load4_guarded(e_tile, pos, ti.len, ev);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            gs[j][c] = __fadd_rn(ev[c], by_n(gs[j][c]));  // v
            xs[j][c] = by_n(xs[j][c]);                    // xbar
        }
        // e' = v - p with p = v
        if (FAST) {
            *reinterpret_cast<float4 *>(e_tile + pos) = make_float4(__fsub_rn(gs[j][0], gs[j][0]), __fsub_rn(gs[j][1], gs[j][1]),
                                                                    __fsub_rn(gs[j][2], gs[j][2]), __fsub_rn(gs[j][3], gs[j][3]));
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (pos + c < ti.len) e_tile[pos + c] = __fsub_rn(gs[j][c], gs[j][c]);
        }
    }
#pragma unroll 4
    for (int i = 0; i < p.N; ++i) {
        const GT *g_tile = g_tile0 + (int64_t)i * p.d;
        float *x_tile = x_tile0 + (int64_t)i * p.d;
#pragma unroll
        for (int j = 0; j < HR; ++j) {
            const int pos = tile_pos(warp, lane, j0 + j);
            float g[4], x[4];
            if (FAST) load4_cached(g_tile + pos, g);
            else load4_guarded(g_tile, pos, ti.len, g);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float diff = __fsub_rn(gs[j][c], g[c]);   // p - p^i, p = v, p^i = g^i
                const float u = __fadd_rn(diff, g[c]);
                x[c] = __fsub_rn(xs[j][c], __fmul_rn(lr, u));
            }
            if (FAST) {
                __stcs(reinterpret_cast<float4 *>(x_tile + pos), make_float4(x[0], x[1], x[2], x[3]));
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (pos + c < ti.len) x_tile[pos + c] = x[c];
            }
        }
    }
}

template <typename GT>
__global__ void __launch_bounds__(THREADS, (sizeof(GT) == 4 ? 2 : 3)) average_step_kernel(const __grid_constant__ Params p, const float lr) {
    const TileInfo ti = locate_tile(p, blockIdx.x);
    // two CTAs share a tile (rows 0-3 and rows 4-7 of every warp's slice): half the accumulators
    // per thread, twice the CTAs in flight
    const int j0 = 4 * blockIdx.y;
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & 3) == 0) && ((p.d & 3) == 0);
    if (fast) average_tile<GT, true>(p, ti, lr, j0);
    else average_tile<GT, false>(p, ti, lr, j0);
}

// xbar = (1/N) sum_i x^i (the ENSURE line of Algorithm 1), one CTA per tile.
template <bool FAST>
__device__ __forceinline__ void mean_tile(const Params &p, const TileInfo &ti, float *out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WorkerDivisor by_n(p.N);
    const float *x_tile0 = p.X + ti.seg_beg + ti.rel;
    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[j][c] = 0.0f;
#pragma unroll 2
    for (int i = 0; i < p.N; ++i) {   // worker order; the 8 rows of a worker are fetched together
        const float *x_tile = x_tile0 + (int64_t)i * p.d;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int pos = tile_pos(warp, lane, j);
            float x[4];
            if (FAST) load4_stream(x_tile + pos, x);
            else load4_guarded(x_tile, pos, ti.len, x);
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[j][c] = __fadd_rn(acc[j][c], x[c]);
        }
    }
    float *o = out + ti.seg_beg + ti.rel;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pos = tile_pos(warp, lane, j);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (pos + c < ti.len) o[pos + c] = by_n(acc[j][c]);
    }
}

__global__ void __launch_bounds__(THREADS) mean_params_kernel(const __grid_constant__ Params p, float *out) {
    const TileInfo ti = locate_tile(p, blockIdx.x);
    // full tile and every worker's row 16-byte aligned: the sweep over the workers carries no branch
    if ((ti.len == TILE) && ((ti.seg_beg & 3) == 0) && ((p.d & 3) == 0)) mean_tile<true>(p, ti, out);
    else mean_tile<false>(p, ti, out);
}

cudaError_t launch_average_step(const Params &p, float lr, cudaStream_t st) {
    const dim3 grid(p.TT, 2);
    if (p.gdt == DT_F32) average_step_kernel<float><<<grid, THREADS, 0, st>>>(p, lr);
    else average_step_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(p, lr);
    return cudaGetLastError();
}

cudaError_t launch_mean_params(const Params &p, float *out, cudaStream_t st) {
    mean_params_kernel<<<p.TT, THREADS, 0, st>>>(p, out);
    return cudaGetLastError();
}

}  // namespace liec
