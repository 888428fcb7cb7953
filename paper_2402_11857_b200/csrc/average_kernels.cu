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

// ------------------------------------------------------------------------------------------------
// The same iteration with the workers' gradients of the CTA's slice held in shared memory between
// the two sweeps, so that g is read from HBM once.  A CTA owns SLICE = 1024 * GROUPS consecutive
// coordinates of a full, 16-byte aligned tile: one thread starts N bulk copies (TMA, one per
// worker's row of the slice, all counted on one mbarrier) and, while they are in flight, every
// thread sums the models in worker order; then the gradients are summed from shared memory, v and
// xbar follow, and the second sweep reads g from shared memory again.  Same operations in the same
// order as average_tile.  Tiles that are ragged or misaligned take average_tile (two of the CTAs).
// Used when N rows of the slice fit the shared memory that keeps two or three CTAs on an SM.
// ------------------------------------------------------------------------------------------------
constexpr size_t AVG_SMEM_LIMIT = 96 * 1024;

template <typename GT, int GROUPS>
__global__ void __launch_bounds__(THREADS) average_step_staged_kernel(const __grid_constant__ Params p, const float lr) {
    constexpr int SLICE = THREADS * 4 * GROUPS;
    constexpr int ALIGN_MASK = sizeof(GT) == 4 ? 3 : 7;   // elements per 16 bytes, minus one
    extern __shared__ __align__(128) unsigned char avg_smem[];
    GT *g_s = reinterpret_cast<GT *>(avg_smem);            // [N][SLICE]
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int copy_ok;
    const TileInfo ti = locate_tile(p, blockIdx.x);
    const bool fast = (ti.len == TILE) && ((ti.seg_beg & ALIGN_MASK) == 0) && ((p.d & ALIGN_MASK) == 0);
    if (!fast) {   // (uniform over the CTA)
        if (blockIdx.y < 2) average_tile<GT, false>(p, ti, lr, 4 * blockIdx.y);
        return;
    }
    const int64_t first = ti.seg_beg + ti.rel + (int64_t)blockIdx.y * SLICE;   // first coordinate of the slice
    const GT *g0 = reinterpret_cast<const GT *>(p.G) + first;
    float *x0 = p.X + first;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint32_t row_bytes = SLICE * sizeof(GT);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     ::"r"(smem_u32(&bar)), "r"(row_bytes * (uint32_t)p.N + p.copy_expect_extra) : "memory");
        for (int i = 0; i < p.N; ++i)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(g_s + (size_t)i * SLICE)), "l"(g0 + (int64_t)i * p.d), "r"(row_bytes), "r"(smem_u32(&bar)) : "memory");
        copy_ok = 1;
    }
    // models in worker order while the gradients arrive
    float xs[GROUPS][4], gs[GROUPS][4];
#pragma unroll
    for (int q = 0; q < GROUPS; ++q)
#pragma unroll
        for (int c = 0; c < 4; ++c) { xs[q][c] = 0.0f; gs[q][c] = 0.0f; }
#pragma unroll 8
    for (int i = 0; i < p.N; ++i) {
#pragma unroll
        for (int q = 0; q < GROUPS; ++q) {
            float x[4];
            load4_stream(x0 + (int64_t)i * p.d + (q * THREADS + threadIdx.x) * 4, x);
#pragma unroll
            for (int c = 0; c < 4; ++c) xs[q][c] = __fadd_rn(xs[q][c], x[c]);
        }
    }
    if (threadIdx.x == 0 && !mbar_wait_bounded(&bar, 0u, p.copy_wait_limit)) {
        atomicOr(p.status, STATUS_COPY_TIMEOUT);
        mbar_drain(&bar, 0u);
        copy_ok = 0;
    }
    __syncthreads();
    if (!copy_ok) return;   // nothing of this slice has been written
    auto g_at = [&](int i, int q, float (&g)[4]) {
        const GT *src = g_s + (size_t)i * SLICE + (q * THREADS + threadIdx.x) * 4;
        if constexpr (sizeof(GT) == 4) {
            const float4 v4 = *reinterpret_cast<const float4 *>(src);
            g[0] = v4.x; g[1] = v4.y; g[2] = v4.z; g[3] = v4.w;
        } else {
            const uint2 v2 = *reinterpret_cast<const uint2 *>(src);
            g[0] = __uint_as_float(v2.x << 16); g[1] = __uint_as_float(v2.x & 0xffff0000u);
            g[2] = __uint_as_float(v2.y << 16); g[3] = __uint_as_float(v2.y & 0xffff0000u);
        }
    };
    for (int i = 0; i < p.N; ++i) {
#pragma unroll
        for (int q = 0; q < GROUPS; ++q) {
            float g[4];
            g_at(i, q, g);
#pragma unroll
            for (int c = 0; c < 4; ++c) gs[q][c] = __fadd_rn(gs[q][c], g[c]);
        }
    }
    const WorkerDivisor by_n(p.N);
    float *e0 = p.e + first;
#pragma unroll
    for (int q = 0; q < GROUPS; ++q) {
        float ev[4];
        float *ep = e0 + (q * THREADS + threadIdx.x) * 4;
        load4_stream(ep, ev);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            gs[q][c] = __fadd_rn(ev[c], by_n(gs[q][c]));  // v
            xs[q][c] = by_n(xs[q][c]);                    // xbar
        }
        // e' = v - p with p = v
        *reinterpret_cast<float4 *>(ep) = make_float4(__fsub_rn(gs[q][0], gs[q][0]), __fsub_rn(gs[q][1], gs[q][1]),
                                                      __fsub_rn(gs[q][2], gs[q][2]), __fsub_rn(gs[q][3], gs[q][3]));
    }
#pragma unroll 4
    for (int i = 0; i < p.N; ++i) {
#pragma unroll
        for (int q = 0; q < GROUPS; ++q) {
            float g[4], x[4];
            g_at(i, q, g);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float diff = __fsub_rn(gs[q][c], g[c]);   // p - p^i, p = v, p^i = g^i
                const float u = __fadd_rn(diff, g[c]);
                x[c] = __fsub_rn(xs[q][c], __fmul_rn(lr, u));
            }
            __stcs(reinterpret_cast<float4 *>(x0 + (int64_t)i * p.d + (q * THREADS + threadIdx.x) * 4), make_float4(x[0], x[1], x[2], x[3]));
        }
    }
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

template <typename GT>
static bool launch_average_staged(const Params &p, float lr, cudaStream_t st) {
    const size_t row1 = (size_t)p.N * THREADS * 4 * sizeof(GT);   // N rows of a 1024-element slice
    if (2 * row1 <= 64 * 1024) {
        average_step_staged_kernel<GT, 2><<<dim3(p.TT, TILE / (THREADS * 8)), THREADS, 2 * row1, st>>>(p, lr);
        return true;
    }
    if (row1 <= AVG_SMEM_LIMIT) {
        average_step_staged_kernel<GT, 1><<<dim3(p.TT, TILE / (THREADS * 4)), THREADS, row1, st>>>(p, lr);
        return true;
    }
    return false;
}

cudaError_t configure_average_kernels() {
    const void *kernels[] = {(const void *)average_step_staged_kernel<float, 1>, (const void *)average_step_staged_kernel<float, 2>,
                             (const void *)average_step_staged_kernel<__nv_bfloat16, 1>, (const void *)average_step_staged_kernel<__nv_bfloat16, 2>};
    cudaError_t e = cudaSuccess;
    for (const void *k : kernels)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AVG_SMEM_LIMIT);
    return e;
}

cudaError_t launch_average_step(const Params &p, float lr, cudaStream_t st) {
    // gradients held in shared memory between the sweeps when N rows of a slice fit
    if (p.gdt == DT_F32 ? launch_average_staged<float>(p, lr, st) : launch_average_staged<__nv_bfloat16>(p, lr, st))
        return cudaGetLastError();
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
