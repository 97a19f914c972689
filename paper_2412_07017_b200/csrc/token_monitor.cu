// Token monitor's hook into next-token selection (paper Section 5.1): a finite-state machine over CML
// (Section 3) decides which tokens a sequence may produce next, [INTR] is never among them (interrupts
// are injected by the system, not generated), the allowed token with the largest logit is taken
// (lowest id among equals; NaN never), and the state machine reports a finished function call, a
// finished trap and whether the sequence is inside a function-call block (the critical section in
// which interrupts are deferred, Section 3.2).
//
// The logits are streamed once (16-byte loads, several CTAs per sequence): the kernel is bound by HBM,
// vocab * element size bytes per sequence.  The mask costs nothing per element: the five CML tokens are
// set aside during the scan and compared at the end according to the state.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>

#include <algorithm>

#include "asynclm.h"
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace {

constexpr int kMonThreads = 256;
constexpr int kMonVecs = 8;                        // 16-byte vectors in flight per thread
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

// (value, id) as one 64-bit key whose unsigned order is "larger value first, then lower id": floats map
// to unsigned integers monotonically (sign bit flipped for positives, all bits for negatives), the id
// goes in complemented.  Key 0 means "nothing yet" (no real candidate maps to it: -NaN patterns never
// enter, and -inf maps to 0x007fffff in the upper half).
__device__ __forceinline__ unsigned long long pack_key(float v, int i) {
    const unsigned u = __float_as_uint(v);
    const unsigned ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)ord << 32) | (unsigned)(0x7fffffff - i);
}
__device__ __forceinline__ Best unpack_key(unsigned long long k) {
    if (k == 0) return Best{-INFINITY, INT_MAX};
    const unsigned ord = (unsigned)(k >> 32);
    const unsigned u = (ord & 0x80000000u) ? (ord & 0x7fffffffu) : ~ord;
    return Best{__uint_as_float(u), 0x7fffffff - (int)(unsigned)(k & 0xffffffffu)};
}

// Grid: (slices, batch).  Every CTA scans one slice of a sequence's row and folds its best ordinary
// token into the row's key with one atomic max; the CTA that arrives last (per-row counter) finishes the
// row: it lets the CML tokens the state allows compete, advances the state machine and puts the two
// workspace words back to zero for the next call.  The result does not depend on arrival order.
template <typename T>
__global__ void __launch_bounds__(kMonThreads)
token_monitor_kernel(const T* __restrict__ logits, int vocab, int64_t row_stride, asynclm_cml_tokens tok,
                     const int32_t* __restrict__ state_in, int32_t* __restrict__ token_out,
                     int32_t* __restrict__ state_out, int32_t* __restrict__ flags_out,
                     unsigned long long* __restrict__ ws) {
    constexpr int VEC = 16 / sizeof(T);
    const int seq = blockIdx.y;
    const T* row = logits + (int64_t)seq * row_stride;
    Best best{-INFINITY, INT_MAX};
    auto offer = [&](float v, int i) {
        // NaN fails both comparisons; the CML tokens take no part in the scan
        if (better(v, i, best) && !is_special(i, tok)) best = Best{v, i};
    };
    const int nvec = vocab / VEC;
    const int per = (nvec + gridDim.x - 1) / gridDim.x;
    const int j_end = min(nvec, (int)(blockIdx.x + 1) * per);
    for (int j0 = blockIdx.x * per + threadIdx.x; j0 < j_end; j0 += kMonVecs * kMonThreads) {
        uint4 w[kMonVecs];
#pragma unroll
        for (int u = 0; u < kMonVecs; ++u) {
            const int j = j0 + u * kMonThreads;
            if (j < j_end) w[u] = ldg_nc_v4(reinterpret_cast<const uint4*>(row) + j);
        }
#pragma unroll
        for (int u = 0; u < kMonVecs; ++u) {
            const int j = j0 + u * kMonThreads;
            if (j >= j_end) break;
            const T* e = reinterpret_cast<const T*>(&w[u]);
            // the vector's largest value first: only a vector that can change the best is looked at
            // element by element (NaN compares false everywhere and drops out of fmaxf)
            float vmax = -INFINITY;
#pragma unroll
            for (int k = 0; k < VEC; ++k) vmax = fmaxf(vmax, to_f32<T>(e[k]));
            if (vmax >= best.v) {
                // (the five CML ids are tested per vector, not per element: a vector that holds none of
                // them, which is nearly every vector, takes the short path)
                const int lo = j * VEC;
                const bool has_special = (unsigned)(tok.call - lo) < VEC || (unsigned)(tok.intr - lo) < VEC ||
                                         (unsigned)(tok.trap - lo) < VEC || (unsigned)(tok.end - lo) < VEC ||
                                         (unsigned)(tok.head - lo) < VEC;
                if (has_special) {
#pragma unroll
                    for (int k = 0; k < VEC; ++k) offer(to_f32<T>(e[k]), lo + k);
                } else {
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        const float v = to_f32<T>(e[k]);
                        if (better(v, lo + k, best)) best = Best{v, lo + k};
                    }
                }
            }
        }
    }
    if (blockIdx.x == gridDim.x - 1)
        for (int i = nvec * VEC + threadIdx.x; i < vocab; i += kMonThreads) offer(to_f32<T>(row[i]), i);
    // CTA-wide best: shuffles inside a warp, shared memory across warps
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
    if (threadIdx.x != 0) return;
    for (int w = 1; w < kMonThreads / 32; ++w)
        if (better(sv[w], si[w], best)) best = Best{sv[w], si[w]};
    unsigned long long* key = ws + 2 * (size_t)seq;
    unsigned* arrived = reinterpret_cast<unsigned*>(key + 1);
    if (best.i != INT_MAX) atomicMax(key, pack_key(best.v, best.i));
    __threadfence();
    if (atomicAdd(arrived, 1u) != gridDim.x - 1) return;
    __threadfence();
    best = unpack_key(atomicExch(key, 0ull));
    *arrived = 0;
    // ---- the state machine: which of the CML tokens compete, and where the chosen token leads
    const int state = state_in[seq];
    Best pick = state == kTrap ? Best{-INFINITY, INT_MAX} : best;      // ordinary tokens: everywhere but in a trap block
    auto compete = [&](int id) {
        const float v = to_f32<T>(row[id]);
        if (better(v, id, pick)) pick = Best{v, id};
    };
    if (state == kText) { compete(tok.call); compete(tok.trap); }
    if (state == kCall) { compete(tok.head); compete(tok.end); }
    if (state == kBody || state == kTrap) compete(tok.end);
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
    token_out[seq] = pick.i;
    state_out[seq] = next;
    flags_out[seq] = flags;
}

}  // namespace

}  // namespace asynclm

extern "C" size_t asynclm_token_monitor_workspace_bytes(int32_t batch) { return batch > 0 ? (size_t)batch * 16 : 0; }

extern "C" int asynclm_token_monitor_step(const void* logits, int32_t dtype, int32_t batch, int32_t vocab,
                                          int64_t row_stride, const asynclm_cml_tokens* tokens,
                                          const int32_t* state_in, int32_t* token_out, int32_t* state_out,
                                          int32_t* flags_out, void* workspace, void* stream) {
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
    if (!logits || !state_in || !token_out || !state_out || !flags_out || !workspace || ((uintptr_t)logits & 15) != 0 ||
        ((uintptr_t)workspace & 15) != 0 || ((size_t)row_stride * esz) % 16 != 0 || batch > 65535)
        return ASYNCLM_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // slices per row: enough CTAs of 32 KB in flight to fill the machine several times over, at least
    // one pass of kMonVecs vectors per thread each
    const int nvec = vocab / (16 / (int)esz);
    const int max_slices = std::max(1, nvec / (kMonThreads * kMonVecs));
    const int slices = std::max(1, std::min(max_slices, (148 * 16 + batch - 1) / batch));
    const dim3 grid((unsigned)slices, (unsigned)batch);
    if (dtype == ASYNCLM_DTYPE_BF16)
        token_monitor_kernel<__nv_bfloat16><<<grid, kMonThreads, 0, s>>>((const __nv_bfloat16*)logits, vocab, row_stride, *tokens,
                                                                         state_in, token_out, state_out, flags_out,
                                                                         (unsigned long long*)workspace);
    else
        token_monitor_kernel<float><<<grid, kMonThreads, 0, s>>>((const float*)logits, vocab, row_stride, *tokens, state_in,
                                                                 token_out, state_out, flags_out, (unsigned long long*)workspace);
    return cuda_status(cudaGetLastError());
}
