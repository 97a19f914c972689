// Launchers of the device kernels (internal).  Each returns a cudaError_t from the launch.
#pragma once
#include <cuda_runtime.h>

#include "plan_types.h"

namespace asynclm {

cudaError_t launch_kv_append(const DevPlan& p, const void* k_new, const void* v_new, void* kv_pool,
                             cudaStream_t stream);

cudaError_t launch_attn_decode(const DevPlan& p, const void* q, const void* kv_pool, void* out,
                               float* lse, cudaStream_t stream);

// Tensor-core (tcgen05) attention for span tiles; head_dim 128 only.
cudaError_t launch_attn_append_tc(const DevPlan& p, const void* q, const void* kv_pool, void* out,
                                  float* lse, cudaStream_t stream);

cudaError_t launch_lse_merge(const DevPlan& p, void* out, float* lse, cudaStream_t stream);

}  // namespace asynclm
