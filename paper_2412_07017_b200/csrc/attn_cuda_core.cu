// CUDA-core attention for decode rows and short spans: one warp per persistent slot.
//
// Each new token of a step attends to its sequence's whole cached context plus the part of its own
// span up to itself (paper Section 3.2 / 5.3: the interrupt tokens are appended to the context and
// processed in the next decoding step).  A work item is one KV chunk of one (sequence, kv head,
// token); the G query heads that share the kv head are processed together so each K/V row is read
// once.  Split contexts write (normalised partial output, log-sum-exp) pairs that lse_merge.cu
// combines.
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

template <int D, int G>
__global__ void __launch_bounds__(128)
attn_cuda_core_kernel(DevPlan p, const __nv_bfloat16* __restrict__ q,
                      const __nv_bfloat16* __restrict__ pool, __nv_bfloat16* __restrict__ out,
                      float* __restrict__ lse) {
    constexpr int LPR = D / 8;        // lanes that share one K/V row (16 bytes each)
    constexpr int TPW = 32 / LPR;     // rows covered by one warp-wide load
    constexpr int U = 4;              // independent row loads in flight per lane and tensor
    const int lane = threadIdx.x & 31;
    const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (slot >= p.num_ctas_cuda) return;
    const int sub = lane % LPR;       // which 8-element slice of the row
    const int grp = lane / LPR;       // which row of the warp-wide load
    const int Hq = p.num_q_heads, Hkv = p.num_kv_heads;
    const float qscale = p.sm_scale * kLog2e;

    for (int ii = p.cta_indptr_cuda[slot]; ii < p.cta_indptr_cuda[slot + 1]; ++ii) {
        const Item it = p.items[ii];
        const Unit u = p.units[it.unit];
        for (int t = 0; t < u.ntok; ++t) {
            const int limit = min(it.kv1, u.kv_limit0 + t);
            const int row = u.q_row0 + t;
            float qf[G][8];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint4 w = *reinterpret_cast<const uint4*>(
                    q + ((size_t)row * Hq + (size_t)u.kv_head * G + g) * D + sub * 8);
                qf[g][0] = bf16_lo(w.x) * qscale; qf[g][1] = bf16_hi(w.x) * qscale;
                qf[g][2] = bf16_lo(w.y) * qscale; qf[g][3] = bf16_hi(w.y) * qscale;
                qf[g][4] = bf16_lo(w.z) * qscale; qf[g][5] = bf16_hi(w.z) * qscale;
                qf[g][6] = bf16_lo(w.w) * qscale; qf[g][7] = bf16_hi(w.w) * qscale;
            }
            float m[G], l[G], o[G][8];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                m[g] = -INFINITY;
                l[g] = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
            }
            for (int base = it.kv0; base < limit; base += TPW * U) {
                uint4 kw[U], vw[U];
                bool valid[U];
#pragma unroll
                for (int x = 0; x < U; ++x) {
                    const int tok = base + x * TPW + grp;
                    valid[x] = tok < limit;
                    kw[x] = make_uint4(0, 0, 0, 0);
                    vw[x] = make_uint4(0, 0, 0, 0);
                    if (valid[x]) {
                        const int64_t page = __ldg(p.page_indices + u.page_base + tok / kPage);
                        const size_t off = pool_row_offset(page, 0, u.kv_head, tok % kPage, Hkv, D) + sub * 8;
                        kw[x] = ldg_nc_v4(pool + off);
                        vw[x] = ldg_nc_v4(pool + off + (size_t)Hkv * kPage * D);
                    }
                }
                float s[U][G];
#pragma unroll
                for (int x = 0; x < U; ++x) {
                    float kf[8] = {bf16_lo(kw[x].x), bf16_hi(kw[x].x), bf16_lo(kw[x].y), bf16_hi(kw[x].y),
                                   bf16_lo(kw[x].z), bf16_hi(kw[x].z), bf16_lo(kw[x].w), bf16_hi(kw[x].w)};
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        float a = 0.f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) a = fmaf(qf[g][e], kf[e], a);
#pragma unroll
                        for (int off = 1; off < LPR; off <<= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
                        s[x][g] = valid[x] ? a : -INFINITY;
                    }
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float mn = m[g];
#pragma unroll
                    for (int x = 0; x < U; ++x) mn = fmaxf(mn, s[x][g]);
                    const float ms = mn == -INFINITY ? 0.f : mn;
                    const float corr = fast_exp2(m[g] - ms);
                    m[g] = mn;
                    l[g] *= corr;
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[g][e] *= corr;
#pragma unroll
                    for (int x = 0; x < U; ++x) s[x][g] = fast_exp2(s[x][g] - ms);
                }
#pragma unroll
                for (int x = 0; x < U; ++x) {
                    float vf[8] = {bf16_lo(vw[x].x), bf16_hi(vw[x].x), bf16_lo(vw[x].y), bf16_hi(vw[x].y),
                                   bf16_lo(vw[x].z), bf16_hi(vw[x].z), bf16_lo(vw[x].w), bf16_hi(vw[x].w)};
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        l[g] += s[x][g];
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[g][e] = fmaf(s[x][g], vf[e], o[g][e]);
                    }
                }
            }
            // combine the TPW row groups of the warp
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float m2 = __shfl_xor_sync(0xffffffffu, m[g], off);
                    const float l2 = __shfl_xor_sync(0xffffffffu, l[g], off);
                    const float mn = fmaxf(m[g], m2);
                    const float ms = mn == -INFINITY ? 0.f : mn;
                    const float c1 = fast_exp2(m[g] - ms), c2 = fast_exp2(m2 - ms);
                    l[g] = l[g] * c1 + l2 * c2;
                    m[g] = mn;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float o2 = __shfl_xor_sync(0xffffffffu, o[g][e], off);
                        o[g][e] = o[g][e] * c1 + o2 * c2;
                    }
                }
            }
            if (grp == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float inv = l[g] > 0.f ? 1.f / l[g] : 0.f;
                    const float lse2 = l[g] > 0.f ? m[g] + log2f(l[g]) : -INFINITY;
                    if (u.partial_base < 0) {
                        const size_t at = ((size_t)row * Hq + (size_t)u.kv_head * G + g) * D + sub * 8;
                        uint4 w;
                        w.x = pack_bf16x2(o[g][0] * inv, o[g][1] * inv);
                        w.y = pack_bf16x2(o[g][2] * inv, o[g][3] * inv);
                        w.z = pack_bf16x2(o[g][4] * inv, o[g][5] * inv);
                        w.w = pack_bf16x2(o[g][6] * inv, o[g][7] * inv);
                        *reinterpret_cast<uint4*>(out + at) = w;
                        if (lse != nullptr && sub == 0)
                            lse[(size_t)row * Hq + (size_t)u.kv_head * G + g] = lse2 * kLn2;
                    } else {
                        const size_t prow = (size_t)u.partial_base + (size_t)it.chunk * u.ntok + t;
                        float4* dst = reinterpret_cast<float4*>(p.partial_o + (prow * G + g) * D + sub * 8);
                        dst[0] = make_float4(o[g][0] * inv, o[g][1] * inv, o[g][2] * inv, o[g][3] * inv);
                        dst[1] = make_float4(o[g][4] * inv, o[g][5] * inv, o[g][6] * inv, o[g][7] * inv);
                        if (sub == 0) p.partial_lse[prow * G + g] = lse2;
                    }
                }
            }
        }
    }
}

template <int D>
static cudaError_t launch_d(const DevPlan& p, const void* q, const void* pool, void* out, float* lse,
                            cudaStream_t stream) {
    const int warps = 4;
    const int blocks = (p.num_ctas_cuda + warps - 1) / warps;
    auto Q = (const __nv_bfloat16*)q;
    auto KV = (const __nv_bfloat16*)pool;
    auto O = (__nv_bfloat16*)out;
    switch (p.group) {
        case 1: attn_cuda_core_kernel<D, 1><<<blocks, warps * 32, 0, stream>>>(p, Q, KV, O, lse); break;
        case 2: attn_cuda_core_kernel<D, 2><<<blocks, warps * 32, 0, stream>>>(p, Q, KV, O, lse); break;
        case 4: attn_cuda_core_kernel<D, 4><<<blocks, warps * 32, 0, stream>>>(p, Q, KV, O, lse); break;
        case 8: attn_cuda_core_kernel<D, 8><<<blocks, warps * 32, 0, stream>>>(p, Q, KV, O, lse); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_attn_cuda_core(const DevPlan& p, const void* q, const void* kv_pool, void* out,
                                  float* lse, cudaStream_t stream) {
    if (p.num_items_cuda == 0) return cudaSuccess;
    if (p.head_dim == 128) return launch_d<128>(p, q, kv_pool, out, lse, stream);
    if (p.head_dim == 64) return launch_d<64>(p, q, kv_pool, out, lse, stream);
    return cudaErrorInvalidValue;
}

}  // namespace asynclm
