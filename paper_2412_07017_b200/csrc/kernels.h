// Launchers of the device kernels (internal).  Each returns a cudaError_t from the launch.
#pragma once
#include <cuda_runtime.h>

#include "plan_types.h"

namespace asynclm {

cudaError_t launch_kv_append(const DevPlan& p, const void* k_new, const void* v_new, void* kv_pool,
                             cudaStream_t stream);

// All attention kernels of a step: span tiles and warp-body items (one fused launch when the step
// has both), writing final rows to `out` and split rows to the plan's partials.  With app.k_new set
// the kernels first put every new K/V row they are about to read into its page slot themselves.
cudaError_t launch_attention(const DevPlan& p, const void* q, const void* kv_pool, void* out, float* lse,
                             cudaStream_t stream, AppendSrc app = AppendSrc{nullptr, nullptr, nullptr});

cudaError_t launch_lse_merge(const DevPlan& p, void* out, float* lse, cudaStream_t stream);

// Remembers `e` as the calling thread's last CUDA error (asynclm_last_cuda_error) and clears the
// runtime's sticky launch error; returns ASYNCLM_OK for cudaSuccess, else ASYNCLM_ERR_CUDA.
int cuda_status(cudaError_t e);

// ASYNCLM_OK if the current device is the one the plan was made for, else ASYNCLM_ERR_INVALID_ARG
// (ASYNCLM_ERR_CUDA if the device cannot be queried).
int check_plan_device(int plan_device);

}  // namespace asynclm
