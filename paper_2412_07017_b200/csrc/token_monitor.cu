// Token monitor's hook into next-token selection (paper Section 5.1): a finite-state machine over CML
// (Section 3) decides which tokens a sequence may produce next, [INTR] is never among them (interrupts
// are injected by the system, not generated), the allowed token with the largest logit is taken
// (lowest id among equals; NaN never), and the state machine reports a finished function call, a
// finished trap and whether the sequence is inside a function-call block (the critical section in
// which interrupts are deferred, Section 3.2).
//
// The logits are streamed once (16-byte loads, several CTAs per sequence): the kernel is bound by HBM,
// vocab * element size bytes per sequence.  The mask costs nothing per element: the scan takes the
// plain maximum, and only a row whose maximum is a token its state forbids is looked at a second time.
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

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    // largest of the 8 values of a 16-byte vector (NaN drops out of max)
    static __device__ __forceinline__ float vmax(const uint4& w) {
        const unsigned u[4] = {w.x, w.y, w.z, w.w};
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < 4; ++k) m = fmaxf(m, fmaxf(bf16_lo(u[k]), bf16_hi(u[k])));
        return m;
    }
    static __device__ __forceinline__ float at(const uint4& w, int k) {
        const unsigned u[4] = {w.x, w.y, w.z, w.w};
        return (k & 1) ? bf16_hi(u[k >> 1]) : bf16_lo(u[k >> 1]);
    }
};
template <> struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ float vmax(const uint4& w) {
        return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)), fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
    }
    static __device__ __forceinline__ float at(const uint4& w, int k) {
        const unsigned u[4] = {w.x, w.y, w.z, w.w};
        return __uint_as_float(u[k]);
    }
};

// Largest element of vectors [j_begin, j_end) of a row (stride of the CTA's threads), lowest id among
// equals; `skip`: leave the five CML tokens out.  Per vector only its maximum is computed; the
// position inside the best vector is found at the end by looking at that one vector again.
template <typename T>
__device__ __forceinline__ Best scan_row(const T* row, int j_begin, int j_end, const asynclm_cml_tokens& tok, bool skip) {
    constexpr int VEC = Vec<T>::N;
    const uint4* v4 = reinterpret_cast<const uint4*>(row);
    float bv = -INFINITY;
    int bj = -1;
    for (int j0 = j_begin + threadIdx.x; j0 < j_end; j0 += kMonVecs * kMonThreads) {
        uint4 w[kMonVecs];
#pragma unroll
        for (int u = 0; u < kMonVecs; ++u) {
            const int j = j0 + u * kMonThreads;
            if (j < j_end) w[u] = ldg_nc_v4(v4 + j);
        }
#pragma unroll
        for (int u = 0; u < kMonVecs; ++u) {
            const int j = j0 + u * kMonThreads;
            if (j >= j_end) break;
            float m = Vec<T>::vmax(w[u]);
            if (skip) {      // (the rare second pass) recompute without the CML tokens this vector may hold
                m = -INFINITY;
#pragma unroll
                for (int k = 0; k < VEC; ++k)
                    if (!is_special(j * VEC + k, tok)) m = fmaxf(m, Vec<T>::at(w[u], k));
            }
            if (m > bv) { bv = m; bj = j; }      // a thread's vectors come in increasing order: the first one wins a tie
        }
    }
    Best best{-INFINITY, INT_MAX};
    if (bj >= 0) {
        const uint4 w = ldg_nc_v4(v4 + bj);
#pragma unroll
        for (int k = VEC - 1; k >= 0; --k)
            if (Vec<T>::at(w, k) == bv && !(skip && is_special(bj * VEC + k, tok))) best = Best{bv, bj * VEC + k};
    }
    return best;
}

// CTA-wide best in thread 0 (shuffles inside a warp, shared memory across warps).
__device__ __forceinline__ Best block_best(Best best, float* sv, int* si) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float v = __shfl_xor_sync(0xffffffffu, best.v, off);
        const int i = __shfl_xor_sync(0xffffffffu, best.i, off);
        if (better(v, i, best)) best = Best{v, i};
    }
    __syncthreads();      // (sv / si may still be read from an earlier call)
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best.v; si[threadIdx.x >> 5] = best.i; }
    __syncthreads();
    if (threadIdx.x == 0)
        for (int w = 1; w < kMonThreads / 32; ++w)
            if (better(sv[w], si[w], best)) best = Best{sv[w], si[w]};
    return best;
}

// Grid: (slices, batch).  Every CTA scans one slice of a sequence's row, ALL tokens alike, and folds its
// best into the row's key with one atomic max; the CTA that arrives last (per-row counter) finishes the
// row.  If the row's largest logit belongs to an ordinary token or to a CML token the state allows, that
// token is the answer (an allowed token that beats everything beats everything allowed).  Only if it
// belongs to a CML token the state forbids, a "hallucinated" [INTR] say, the last CTA scans the row once
// more without the CML tokens and lets the allowed ones compete.  Then the state machine advances and
// the two workspace words go back to zero.  The result does not depend on arrival order.
template <typename T>
__global__ void __launch_bounds__(kMonThreads)
token_monitor_kernel(const T* __restrict__ logits, int vocab, int64_t row_stride, asynclm_cml_tokens tok,
                     const int32_t* __restrict__ state_in, int32_t* __restrict__ token_out,
                     int32_t* __restrict__ state_out, int32_t* __restrict__ flags_out,
                     unsigned long long* __restrict__ ws) {
    constexpr int VEC = Vec<T>::N;
    __shared__ float sv[kMonThreads / 32];
    __shared__ int si[kMonThreads / 32];
    __shared__ int s_rescan;
    const int seq = blockIdx.y;
    const T* row = logits + (int64_t)seq * row_stride;
    if (state_in[seq] == kTrap) {
        // [TRAP] is followed by [END] whatever the logits say: nothing to read
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            token_out[seq] = tok.end;
            state_out[seq] = kText;
            flags_out[seq] = ASYNCLM_MONITOR_TRAP;
        }
        return;
    }
    const int nvec = vocab / VEC;
    const int per = (nvec + gridDim.x - 1) / gridDim.x;
    Best best = scan_row<T>(row, blockIdx.x * per, min(nvec, (int)(blockIdx.x + 1) * per), tok, false);
    if (blockIdx.x == gridDim.x - 1)      // the row's ragged end, element by element
        for (int i = nvec * VEC + threadIdx.x; i < vocab; i += kMonThreads) {
            const float v = to_f32<T>(row[i]);
            if (better(v, i, best)) best = Best{v, i};
        }
    best = block_best(best, sv, si);
    unsigned long long* key = ws + 2 * (size_t)seq;
    unsigned* arrived = reinterpret_cast<unsigned*>(key + 1);
    const int state = state_in[seq];
    auto allowed_special = [&](int id) {
        return (state == kText && (id == tok.call || id == tok.trap)) || (state == kCall && (id == tok.head || id == tok.end)) ||
               ((state == kBody || state == kTrap) && id == tok.end);
    };
    if (threadIdx.x == 0) {
        s_rescan = -1;      // -1: this CTA is not the last one of its row
        if (best.i != INT_MAX) atomicMax(key, pack_key(best.v, best.i));
        __threadfence();
        if (atomicAdd(arrived, 1u) == gridDim.x - 1) {
            __threadfence();
            best = unpack_key(atomicExch(key, 0ull));
            *arrived = 0;
            const bool ordinary = best.i != INT_MAX && !is_special(best.i, tok);
            // ordinary tokens are allowed everywhere but in a trap block
            const bool settled = best.i != INT_MAX && best.v > -INFINITY &&
                                 (ordinary ? state != kTrap : allowed_special(best.i));
            s_rescan = settled ? 0 : 1;
        }
    }
    __syncthreads();
    if (s_rescan < 0) return;
    if (s_rescan == 1) {
        // the row's best ordinary token (none in a trap block), then the CML tokens the state allows
        Best ord{-INFINITY, INT_MAX};
        if (state != kTrap) {
            ord = scan_row<T>(row, 0, nvec, tok, true);
            for (int i = nvec * VEC + threadIdx.x; i < vocab; i += kMonThreads) {
                const float v = to_f32<T>(row[i]);
                if (!is_special(i, tok) && better(v, i, ord)) ord = Best{v, i};
            }
        }
        ord = block_best(ord, sv, si);
        if (threadIdx.x == 0) {
            best = ord;
            const int ids[5] = {tok.call, tok.trap, tok.head, tok.end, tok.intr};
            for (int a = 0; a < 5; ++a)
                if (allowed_special(ids[a])) {
                    const float v = to_f32<T>(row[ids[a]]);
                    if (better(v, ids[a], best)) best = Best{v, ids[a]};
                }
        }
    }
    if (threadIdx.x != 0) return;
    Best pick = best;
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
    // slices per row: about two CTAs per SM in all, at least one pass of kMonVecs vectors per thread each.
    // Fewer, longer CTAs measure faster than many short ones (256 rows of 128 256 bf16: 20.5 us with one
    // or two slices per row, 22.6 with three or four, 24.7 with five to seven): every CTA ends on a
    // block-wide reduction, an atomic and a fence.
    const int nvec = vocab / (16 / (int)esz);
    const int max_slices = std::max(1, nvec / (kMonThreads * kMonVecs));
    const int slices = std::max(1, std::min(max_slices, (148 * 2 + batch - 1) / batch));
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
