// Launchers of the CUDA kernels (one translation unit per kernel family).
#pragma once
#include <cuda_runtime.h>

#include "plan.h"

namespace liec {

// scaled sign
cudaError_t launch_sign_uplink(const Params &p, cudaStream_t st);
cudaError_t launch_scale_finalize(const Params &p, bool uplink, cudaStream_t st);
cudaError_t launch_server_dense(const Params &p, cudaStream_t st);
cudaError_t launch_sign_error(const Params &p, cudaStream_t st);
cudaError_t launch_identity_downlink(const Params &p, cudaStream_t st);

// top-k (launch counters are bumped per kernel)
cudaError_t launch_topk_hist1(const Params &p, bool uplink, cudaStream_t st, int64_t *launches);
cudaError_t launch_topk_select(const Params &p, bool uplink, cudaStream_t st, int64_t *launches);
cudaError_t launch_topk_small_segments(const Params &p, bool uplink, cudaStream_t st, int64_t *launches);
cudaError_t launch_server_topk(const Params &p, cudaStream_t st, int64_t *launches);
cudaError_t configure_topk_kernels();  // opt-in shared memory sizes; call once per device

// random-k: messages gathered at the caller's subsets, per-tile offsets into them
cudaError_t launch_randk_compress(const Params &p, bool uplink, cudaStream_t st, int64_t *launches);

// model-averaging iteration and mean model
cudaError_t launch_average_step(const Params &p, float lr, cudaStream_t st);
cudaError_t launch_mean_params(const Params &p, float *out, cudaStream_t st);
cudaError_t configure_average_kernels();  // opt-in shared memory sizes; call once per device

// squared norms (monitoring)
cudaError_t launch_sumsq(const Params &p, const void *src, int64_t row_stride, int rows, bool bf16, cudaStream_t st);
cudaError_t launch_sum_finalize(const Params &p, const double *partials, int rows, double *out, cudaStream_t st);

// worker update
cudaError_t launch_worker_update(const Params &p, float lr, cudaStream_t st);

}  // namespace liec
