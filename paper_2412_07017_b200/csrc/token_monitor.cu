// Token monitor's hook into next-token selection (paper Section 5.1): a finite-state machine over CML
// (Section 3) decides which tokens a sequence may produce next, [INTR] is never among them (interrupts
// are injected by the system, not generated), the allowed token with the largest logit is taken
// (lowest id among equals; NaN never), and the state machine reports a finished function call, a
// finished trap and whether the sequence is inside a function-call block (the critical section in
// which interrupts are deferred, Section 3.2).
//
// One CTA per sequence streams the sequence's row of logits once (16-byte loads): the kernel is bound by
// HBM, vocab * element size bytes per sequence.  The mask costs nothing per element: the five CML
// tokens are set aside during the scan and compared at the end according to the state.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>

#include "asynclm.h"
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace {

constexpr int kMonThreads = 1024;
enum { kText = 0, kCall = 1, kBody = 2, kTrap = 3 };

struct Best {
    float v;
    int i;
};
__device__ __forceinline__ bool better(float v, int i, const Best& b) { return v > b.v || (v == b.v && i < b.i); }

__device__ __forceinline__ bool is_special(int i, const asynclm_cml_tokens& t) {
    return i == t.call || i == t.intr || i == t.trap || i == t.end || i == t.head;
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__global__ void __launch_bounds__(kMonThreads)
token_monitor_kernel(const T* __restrict__ logits, int vocab, int64_t row_stride, asynclm_cml_tokens tok,
                     const int32_t* __restrict__ state_in, int32_t* __restrict__ token_out,
                     int32_t* __restrict__ state_out, int32_t* __restrict__ flags_out) {
    constexpr int VEC = 16 / sizeof(T);
    const T* row = logits + (int64_t)blockIdx.x * row_stride;
    Best best{-INFINITY, INT_MAX};
    auto offer = [&](float v, int i) {
        // NaN fails both comparisons; the CML tokens take no part in the scan
        if (better(v, i, best) && !is_special(i, tok)) best = Best{v, i};
    };
    const int nvec = vocab / VEC;
    for (int j = threadIdx.x; j < nvec; j += kMonThreads) {
        const uint4 w = ldg_nc_v4(reinterpret_cast<const uint4*>(row) + j);
        const T* e = reinterpret_cast<const T*>(&w);
#pragma unroll
        for (int k = 0; k < VEC; ++k) offer(to_f32<T>(e[k]), j * VEC + k);
    }
    for (int i = nvec * VEC + threadIdx.x; i < vocab; i += kMonThreads) offer(to_f32<T>(row[i]), i);
    // block-wide best: shuffles inside a warp, shared memory across warps
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float v = __shfl_xor_sync(0xffffffffu, best.v, off);
        const int i = __shfl_xor_sync(0xffffffffu, best.i, off);
        if (better(v, i, best)) best = Best{v, i};
    }
    __shared__ float sv[kMonThreads / 32];
    __shared__ int si[kMonThreads / 32];
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best.v; si[threadIdx.x >> 5] = best.i; }
    __syncthreads();
    if (threadIdx.x >= 32) return;
    best = Best{sv[threadIdx.x], si[threadIdx.x]};
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float v = __shfl_xor_sync(0xffffffffu, best.v, off);
        const int i = __shfl_xor_sync(0xffffffffu, best.i, off);
        if (better(v, i, best)) best = Best{v, i};
    }
    if (threadIdx.x != 0) return;
    // ---- the state machine: which of the CML tokens compete, and where the chosen token leads
    const int state = state_in[blockIdx.x];
    Best pick = state == kTrap ? Best{-INFINITY, INT_MAX} : best;      // ordinary tokens: everywhere but in a trap block
    auto compete = [&](int id) {
        const float v = to_f32<T>(row[id]);
        if (better(v, id, pick)) pick = Best{v, id};
    };
    if (state == kText) { compete(tok.call); compete(tok.trap); }
    if (state == kCall) { compete(tok.head); compete(tok.end); }
    if (state == kBody) compete(tok.end);
    if (pick.i == INT_MAX || pick.v == -INFINITY) {
        // no allowed token has a logit above -inf (all NaN or -inf): the lowest allowed id is taken
        int low = 0;
        while (is_special(low, tok)) ++low;      // lowest ordinary id
        if (state == kText) low = min(low, min(tok.call, tok.trap));
        if (state == kCall) low = min(low, min(tok.head, tok.end));
        if (state == kBody) low = min(low, tok.end);
        if (state == kTrap) low = tok.end;
        pick.i = low;
    }
    int next = state, flags = 0;
    if (state == kText) next = pick.i == tok.call ? kCall : pick.i == tok.trap ? kTrap : kText;
    else if (state == kTrap) { next = kText; flags = ASYNCLM_MONITOR_TRAP; }
    else if (pick.i == tok.end) { next = kText; flags = ASYNCLM_MONITOR_CALL; }
    else if (state == kCall && pick.i == tok.head) next = kBody;
    if (next == kCall || next == kBody) flags |= ASYNCLM_MONITOR_CRITICAL;
    token_out[blockIdx.x] = pick.i;
    state_out[blockIdx.x] = next;
    flags_out[blockIdx.x] = flags;
}

}  // namespace

}  // namespace asynclm

extern "C" int asynclm_token_monitor_step(const void* logits, int32_t dtype, int32_t batch, int32_t vocab,
                                          int64_t row_stride, const asynclm_cml_tokens* tokens,
                                          const int32_t* state_in, int32_t* token_out, int32_t* state_out,
                                          int32_t* flags_out, void* stream) {
    using namespace asynclm;
    if (batch < 0 || vocab <= 5 || !tokens || row_stride < vocab || (dtype != ASYNCLM_DTYPE_BF16 && dtype != ASYNCLM_DTYPE_F32))
        return ASYNCLM_ERR_INVALID_ARG;
    if (batch == 0) return ASYNCLM_OK;
    const int ids[5] = {tokens->call, tokens->intr, tokens->trap, tokens->end, tokens->head};
    for (int a = 0; a < 5; ++a) {
        if (ids[a] < 0 || ids[a] >= vocab) return ASYNCLM_ERR_INVALID_ARG;
        for (int b = 0; b < a; ++b) if (ids[a] == ids[b]) return ASYNCLM_ERR_INVALID_ARG;
    }
    const size_t esz = dtype == ASYNCLM_DTYPE_BF16 ? 2 : 4;
    if (!logits || !state_in || !token_out || !state_out || !flags_out || ((uintptr_t)logits & 15) != 0 ||
        ((size_t)row_stride * esz) % 16 != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (dtype == ASYNCLM_DTYPE_BF16)
        token_monitor_kernel<__nv_bfloat16><<<batch, kMonThreads, 0, s>>>((const __nv_bfloat16*)logits, vocab, row_stride,
                                                                          *tokens, state_in, token_out, state_out, flags_out);
    else
        token_monitor_kernel<float><<<batch, kMonThreads, 0, s>>>((const float*)logits, vocab, row_stride, *tokens,
                                                                  state_in, token_out, state_out, flags_out);
    return cuda_status(cudaGetLastError());
}
