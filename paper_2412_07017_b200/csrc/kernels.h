// Launchers of the device kernels (internal).  Each returns a cudaError_t from the launch.
#pragma once
#include <cuda_runtime.h>

#include "plan_types.h"

namespace asynclm {

cudaError_t launch_kv_append(const DevPlan& p, const void* k_new, const void* v_new, void* kv_pool,
                             cudaStream_t stream);

// All attention kernels of a step: tensor-core span tiles and CUDA-core decode rows (one fused
// launch when the step has both), writing final rows to `out` and split rows to the plan's partials.
cudaError_t launch_attention(const DevPlan& p, const void* q, const void* kv_pool, void* out, float* lse,
                             cudaStream_t stream);

cudaError_t launch_lse_merge(const DevPlan& p, void* out, float* lse, cudaStream_t stream);

}  // namespace asynclm
