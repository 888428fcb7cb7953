// Scaled-sign compression of one vector without any caller-provided or allocated scratch.
//
// The regular path keeps its per-tile partial sums in the caller's workspace.  This entry
// point serves callers that cannot provide one: the partial sums live in a fixed array that
// is part of the library image on every GPU that loads it (64 KiB, held until the process
// exits).  The arithmetic is the same as in the regular uplink pass (same tree, same words).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/liec.h"
#include "device_common.cuh"

namespace liec {

constexpr int64_t NOALLOC_MAX_ELEMENTS = LIEC_NOALLOC_MAX_ELEMENTS;
constexpr int NOALLOC_MAX_TILES = (int)(NOALLOC_MAX_ELEMENTS / TILE);

// One binary64 partial per tile.  Shared by every call on this GPU; it keeps the last call's
// values, which is harmless because a call only reads the partials that it has just written.
static __device__ __align__(256) double g_noalloc_partials[NOALLOC_MAX_TILES];

// One CTA per tile: the same tile routine as the regular uplink pass, partials into the fixed array.
template <typename GT>
__global__ void __launch_bounds__(THREADS) sign_noalloc_kernel(const GT *x, int64_t n, uint32_t *words,
                                                                double *partials) {
    __shared__ double warp_sums[8];
    const int64_t rel = (int64_t)blockIdx.x * TILE;
    const int64_t left = n - rel;
    const int len = left < TILE ? (int)left : TILE;
    // x itself is 16-byte aligned (checked on the host), hence every full tile is
    const double s = sign_tile(x + rel, len, len == TILE, words + rel / 32, warp_sums);
    if (threadIdx.x == 0) partials[blockIdx.x] = s;
}

// Single CTA: tile partials -> ||x||_1 in tree order (the regular path's reducer) -> scale.
__global__ void __launch_bounds__(THREADS) scale_noalloc_kernel(const double *partials, int ntiles, int64_t n,
                                                                 float *scale) {
    __shared__ double buf[FIN_CHUNK];
    __shared__ double chunk_sums[FIN_MAX_CHUNKS];
    const double total = tree_reduce_partials(partials, ntiles, buf, chunk_sums);
    if (threadIdx.x == 0) *scale = __double2float_rn(__ddiv_rn(total, (double)n));
}

// Device address of the scratch array, looked up once per device.  In host code the array's
// name only stands for the symbol; kernels need the address that the runtime reports.
static std::mutex g_noalloc_mutex;
static double *g_noalloc_ptr[64] = {nullptr};

static cudaError_t noalloc_scratch(double **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_partials);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = static_cast<double *>(ptr);
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

}  // namespace liec

static thread_local char g_noalloc_error[256] = "";

extern "C" const char *liec_noalloc_last_error(void) { return g_noalloc_error; }

extern "C" liec_status liec_sign_compress_noalloc(const void *x, int32_t dtype, int64_t n, uint32_t *words,
                                                  float *scale, void *stream) {
    using namespace liec;
    auto bail = [](liec_status st, const char *text) {
        snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", text);
        return st;
    };
    if (!x || !words || !scale) return bail(LIEC_ERR_INVALID_ARG, "x, words and scale must be non-NULL");
    if (reinterpret_cast<uintptr_t>(x) & 15u) return bail(LIEC_ERR_INVALID_ARG, "x must be 16-byte aligned");
    if (dtype != LIEC_F32 && dtype != LIEC_BF16) return bail(LIEC_ERR_INVALID_ARG, "unknown dtype");
    if (n < 1) return bail(LIEC_ERR_INVALID_ARG, "n must be >= 1");
    if (n > NOALLOC_MAX_ELEMENTS) {
        snprintf(g_noalloc_error, sizeof(g_noalloc_error),
                 "n = %lld exceeds LIEC_NOALLOC_MAX_ELEMENTS = %lld (fixed built-in scratch); use liec_uplink_compress",
                 (long long)n, (long long)NOALLOC_MAX_ELEMENTS);
        return LIEC_ERR_UNSUPPORTED;
    }
    double *partials = nullptr;
    cudaError_t e = noalloc_scratch(&partials);
    if (e != cudaSuccess) {
        snprintf(g_noalloc_error, sizeof(g_noalloc_error), "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        return LIEC_ERR_CUDA;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int ntiles = (int)((n + TILE - 1) / TILE);
    if (dtype == LIEC_F32)
        sign_noalloc_kernel<float><<<ntiles, THREADS, 0, st>>>(static_cast<const float *>(x), n, words, partials);
    else
        sign_noalloc_kernel<__nv_bfloat16><<<ntiles, THREADS, 0, st>>>(static_cast<const __nv_bfloat16 *>(x), n, words, partials);
    e = cudaGetLastError();
    if (e == cudaSuccess) {
        scale_noalloc_kernel<<<1, THREADS, 0, st>>>(partials, ntiles, n, scale);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        snprintf(g_noalloc_error, sizeof(g_noalloc_error), "kernel launch failed: %s", cudaGetErrorString(e));
        return LIEC_ERR_CUDA;
    }
    return LIEC_OK;
}
