// C ABI entry points that launch kernels (see include/asynclm.h for the contract).
#include <cuda_runtime.h>

#include "asynclm.h"
#include "kernels.h"
#include "plan_internal.h"

using namespace asynclm;

static thread_local cudaError_t g_last_cuda_error = cudaSuccess;

int asynclm::cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return ASYNCLM_OK;
    g_last_cuda_error = e;
    (void)cudaGetLastError();   // clear the sticky launch-configuration error, if that is what it was
    return ASYNCLM_ERR_CUDA;
}

int asynclm::check_plan_device(int plan_device) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_status(e);
    return dev == plan_device ? ASYNCLM_OK : ASYNCLM_ERR_INVALID_ARG;
}

extern "C" int asynclm_version(void) { return 100; }

extern "C" const char* asynclm_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

extern "C" const char* asynclm_strerror(int status) {
    switch (status) {
        case ASYNCLM_OK: return "ok";
        case ASYNCLM_ERR_INVALID_ARG: return "invalid argument";
        case ASYNCLM_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case ASYNCLM_ERR_PAGE_TABLE: return "page table does not cover a sequence or holds an id outside the pool";
        case ASYNCLM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case ASYNCLM_ERR_CUDA: return "CUDA runtime error";
        case ASYNCLM_ERR_ARCH: return "device is not compute capability 10.x";
        case ASYNCLM_ERR_DEVICE_STATUS: return "a kernel reported a bounded wait that ran out";
        case ASYNCLM_ERR_STATIC_SCRATCH_TOO_SMALL:
            return "the plan's split-KV partial results do not fit the library's fixed scratch array";
        default: return "unknown status";
    }
}

// Longest span for which asynclm_step appends inside the attention kernel.
constexpr int kStepFusedMaxSpan = 64;

static bool runnable(const asynclm_plan_t* plan) {
    return plan && plan->magic == kPlanMagic && !plan->host_only;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

extern "C" int asynclm_kv_append(const asynclm_plan_t* plan, const void* k_new, const void* v_new,
                                 void* kv_pool, void* stream) {
    if (!runnable(plan)) return ASYNCLM_ERR_INVALID_ARG;
    if (plan->dev.total_q == 0) return ASYNCLM_OK;
    if (!k_new || !v_new || !kv_pool || !aligned16(k_new) || !aligned16(v_new) || !aligned16(kv_pool))
        return ASYNCLM_ERR_INVALID_ARG;
    if (int rc = check_plan_device(plan->device)) return rc;
    return cuda_status(launch_kv_append(plan->dev, k_new, v_new, kv_pool, (cudaStream_t)stream));
}

extern "C" int asynclm_attn_mixed(const asynclm_plan_t* plan, const void* q, const void* kv_pool,
                                  void* out, float* lse, void* stream) {
    if (!runnable(plan)) return ASYNCLM_ERR_INVALID_ARG;
    if (plan->dev.total_q == 0) return ASYNCLM_OK;
    if (!q || !kv_pool || !out || !aligned16(q) || !aligned16(kv_pool) || !aligned16(out))
        return ASYNCLM_ERR_INVALID_ARG;
    if (int rc = check_plan_device(plan->device)) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    int rc = cuda_status(launch_attention(plan->dev, q, kv_pool, out, lse, s));
    if (rc != ASYNCLM_OK) return rc;
    return cuda_status(launch_lse_merge(plan->dev, out, lse, s));
}

extern "C" int asynclm_step(const asynclm_plan_t* plan, const void* q, const void* k_new, const void* v_new,
                            void* kv_pool, void* out, float* lse, void* stream) {
    if (!runnable(plan)) return ASYNCLM_ERR_INVALID_ARG;
    if (plan->dev.total_q == 0) return ASYNCLM_OK;
    if (!q || !k_new || !v_new || !kv_pool || !out || !aligned16(q) || !aligned16(k_new) || !aligned16(v_new) ||
        !aligned16(kv_pool) || !aligned16(out))
        return ASYNCLM_ERR_INVALID_ARG;
    if (int rc = check_plan_device(plan->device)) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    int rc;
    if (plan->max_q_len > kStepFusedMaxSpan) {
        // In the fused kernel every item copies the new rows it reads, so the units of one long span
        // copy its first rows again and again (quadratic in the span length): beyond a few hundred
        // tokens the separate append kernel, which copies every row once, is the better first half.
        rc = cuda_status(launch_kv_append(plan->dev, k_new, v_new, kv_pool, s));
        if (rc != ASYNCLM_OK) return rc;
        rc = cuda_status(launch_attention(plan->dev, q, kv_pool, out, lse, s));
    } else {
        rc = cuda_status(launch_attention(plan->dev, q, kv_pool, out, lse, s, AppendSrc{k_new, v_new, kv_pool}));
    }
    if (rc != ASYNCLM_OK) return rc;
    return cuda_status(launch_lse_merge(plan->dev, out, lse, s));
}

#ifdef ASYNCLM_DEBUG
// Checked build only (not part of the public header): the span body's K producer of CTA 0 will not hand
// over its tile-th K tile (1-based; 0 switches it off) in the launches that follow.  The waits that depend
// on that tile (the MMA warp's for the tile, a softmax group's for its scores, the producers' for a free
// slot) then run out after their cycle budget (about a second); the first to do so records its code
// (11, 12, 21, 24, 26 or 31), every role of the CTA leaves through the common exit, tensor memory is
// released and asynclm_last_device_status reports the code.  The GPU neither faults nor hangs: this is
// the test of the bounded waits.  The CTA's output rows are undefined in such a launch.
extern "C" int asynclm_debug_stall_span_tile(asynclm_plan_t* plan, int32_t tile) {
    if (!plan || plan->magic != asynclm::kPlanMagic || tile < 0) return ASYNCLM_ERR_INVALID_ARG;
    plan->dev.debug_stall_tile = tile;
    return ASYNCLM_OK;
}
#endif

extern "C" int asynclm_last_device_status(const asynclm_plan_t* plan, void* stream, int32_t* host_out) {
    if (!runnable(plan) || !host_out) return ASYNCLM_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(host_out, plan->dev.status, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return ASYNCLM_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ASYNCLM_ERR_CUDA;
    return *host_out == 0 ? ASYNCLM_OK : ASYNCLM_ERR_DEVICE_STATUS;
}
