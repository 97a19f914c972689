// asynclm_attn_mixed_static: the attention call for callers that cannot give the library a device
// buffer for split-KV partial results.
//
// Who needs this: code that runs where device allocation is off the table.  Examples are a serving
// loop that has handed every byte of HBM to its KV pool and weight arena at start-up and has no
// allocator left to ask, a plug-in running inside a host process whose memory pool it may not
// touch, and a real-time path in which cudaMalloc is forbidden because it may synchronise the whole
// device.  For them the fp32 partial outputs of split contexts, which are the only scratch memory the
// attention kernels use, live in the fixed array below instead of the plan's device workspace (whose
// size asynclm_plan still checks against the full requirement; that part of it is simply left alone).
//
// The array is part of the library image: every GPU that loads the library carries it from the
// first use of the library on that GPU until the process exits.
#include <cuda_runtime.h>

#include <mutex>

#include "asynclm.h"
#include "kernels.h"
#include "plan_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = ASYNCLM_STATIC_SCRATCH_BYTES;

// Partial outputs ([rows][G][d] fp32) followed, at the next 256-byte boundary, by their
// log-sum-exps ([rows][G] fp32).  Shared by all calls on a device; never needs clearing because
// every partial row the merge reads was written by the attention kernel of the same call.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device.  The symbol's name is only a handle on the
// host; the address a kernel may use has to be asked for, once per device, with that device
// current.
cudaError_t scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int asynclm_attn_mixed_static(const asynclm_plan_t* plan, const void* q,
                                         const void* kv_pool, void* out, float* lse, void* stream) {
    using namespace asynclm;
    if (!plan || plan->magic != kPlanMagic || plan->host_only) return ASYNCLM_ERR_INVALID_ARG;
    if (plan->dev.total_q == 0) return ASYNCLM_OK;
    if (!q || !kv_pool || !out || (((uintptr_t)q | (uintptr_t)kv_pool | (uintptr_t)out) & 15) != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    const size_t rows = (size_t)plan->info.partial_rows;
    const size_t o_bytes = align256(rows * (size_t)plan->dev.group * (size_t)plan->dev.head_dim * sizeof(float));
    const size_t l_bytes = align256(rows * (size_t)plan->dev.group * sizeof(float));
    if (o_bytes + l_bytes > kStaticScratchBytes) return ASYNCLM_ERR_STATIC_SCRATCH_TOO_SMALL;
    if (int rc = check_plan_device(plan->device)) return rc;
    void* base = nullptr;
    if (int rc = cuda_status(scratch_address(&base))) return rc;
    DevPlan d = plan->dev;                       // same plan, partial results redirected
    d.partial_o = (float*)base;
    d.partial_lse = (float*)((unsigned char*)base + o_bytes);
    cudaStream_t s = (cudaStream_t)stream;
    if (int rc = cuda_status(launch_attention(d, q, kv_pool, out, lse, s))) return rc;
    return cuda_status(launch_lse_merge(d, out, lse, s));
}

extern "C" size_t asynclm_static_scratch_bytes(void) { return kStaticScratchBytes; }
