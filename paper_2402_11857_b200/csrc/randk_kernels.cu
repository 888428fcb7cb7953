// Random-k (Def. 3): C(x) keeps the entries of a k_t-subset of every segment; the subset is drawn by
// the caller and arrives as a sorted index list.  Compression is then a gather: the message is the
// index list itself plus the values found there (top-k layout, so that the server pass and the
// worker update consume it unchanged).  For the downlink the kept entries of the error become +0
// (e' = v - p with p = v there).  A second small kernel finds, for every tile, where its entries
// start in the list: the consumers walk the list tile by tile.
#include "device_common.cuh"
#include "kernels.h"

namespace liec {

static_assert(THREADS == TILE_WORDS, "the worker update clears its subset mask with one word per thread");

// First position in the ascending a[lo..hi) whose value is >= key (hi when there is none).
__device__ __forceinline__ int64_t lower_bound_u32(const uint32_t *a, int64_t lo, int64_t hi, uint32_t key) {
    while (lo < hi) {
        const int64_t mid = lo + ((hi - lo) >> 1);
        if (a[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// grid (ceil(K / THREADS), rows): entry q of row r.
//   sets [rows][K] the caller's subsets; src row r at src + r * row_stride (elements of GT);
//   idx_out / val_out [rows][K]; zero_out (downlink only): the array whose kept entries become +0.
template <typename GT>
__global__ void __launch_bounds__(THREADS) randk_gather_kernel(const __grid_constant__ Params p, const uint32_t *sets,
                                                               const GT *src, int64_t row_stride, uint32_t *idx_out,
                                                               float *val_out, float *zero_out) {
    const int64_t q = (int64_t)blockIdx.x * THREADS + threadIdx.x;
    if (q >= p.K) return;
    const int row = blockIdx.y;
    // segment of entry q: last t with k_off[t] <= q
    int lo = 0, hi = p.T;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(p.k_off + mid) <= q) lo = mid; else hi = mid;
    }
    const int t = lo;
    const int64_t seg_beg = __ldg(p.seg_off + t), seg_end = __ldg(p.seg_off + t + 1);
    const uint32_t *set = sets + (int64_t)row * p.K;
    const uint32_t j = set[q];
    bool ok = (int64_t)j >= seg_beg && (int64_t)j < seg_end;
    if (q > __ldg(p.k_off + t) && set[q - 1] >= j) ok = false;  // strictly ascending inside the segment
    float v = 0.0f;
    if (ok) {
        v = load1(src + (int64_t)row * row_stride + j);
        if (zero_out) zero_out[j] = 0.0f;
    } else {
        atomicOr(p.status, (int)STATUS_BAD_SUBSET);
    }
    idx_out[(int64_t)row * p.K + q] = j;  // consumers bound every use of an index by its tile
    val_out[(int64_t)row * p.K + q] = v;
}

// grid (ceil(TT / THREADS), rows): outbase[row][tile] = position in the row's list of the first
// entry at or after the tile's first element.
__global__ void __launch_bounds__(THREADS) randk_outbase_kernel(const __grid_constant__ Params p, const uint32_t *sets,
                                                                uint32_t *outbase) {
    const int tile = blockIdx.x * THREADS + threadIdx.x;
    if (tile >= p.TT) return;
    const int row = blockIdx.y;
    const int t = __ldg(p.tile_seg + tile);
    const int64_t tile_first = __ldg(p.seg_off + t) + (int64_t)(tile - __ldg(p.tile_prefix + t)) * TILE;
    const uint32_t *set = sets + (int64_t)row * p.K;
    const int64_t pos = lower_bound_u32(set, __ldg(p.k_off + t), __ldg(p.k_off + t + 1), (uint32_t)tile_first);
    outbase[(int64_t)row * (p.TT + 1) + tile] = (uint32_t)pos;
}

cudaError_t launch_randk_compress(const Params &p, bool uplink, cudaStream_t st, int64_t *launches) {
    const int rows = uplink ? p.N : 1;
    const uint32_t *sets = uplink ? p.up_sets : p.down_set;
    uint32_t *idx = uplink ? p.up_idx : p.down_idx;
    float *val = uplink ? p.up_val : p.down_val;
    uint32_t *outbase = uplink ? p.up_outbase : p.down_outbase;
    const dim3 g_entries((unsigned)((p.K + THREADS - 1) / THREADS), rows), g_tiles((p.TT + THREADS - 1) / THREADS, rows);
    if (uplink && p.gdt == DT_BF16)
        randk_gather_kernel<__nv_bfloat16><<<g_entries, THREADS, 0, st>>>(p, sets, reinterpret_cast<const __nv_bfloat16 *>(p.G), p.d, idx, val, nullptr);
    else if (uplink)
        randk_gather_kernel<float><<<g_entries, THREADS, 0, st>>>(p, sets, reinterpret_cast<const float *>(p.G), p.d, idx, val, nullptr);
    else  // the error buffer holds v: p = C(v), e' = v - p
        randk_gather_kernel<float><<<g_entries, THREADS, 0, st>>>(p, sets, p.e, 0, idx, val, p.e);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    ++*launches;
    randk_outbase_kernel<<<g_tiles, THREADS, 0, st>>>(p, sets, outbase);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    ++*launches;
    return cudaSuccess;
}

}  // namespace liec
