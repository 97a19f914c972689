// Interrupt append with the rotary position embedding fused in: the form the append takes in a
// multi-layer model of the Llama family (the models the paper serves, Section 6), where a key is
// rotated by its position before it is cached.  New token i of sequence b sits at position ctx_b + i
// (Section 3.2: the block goes to the end of the context).  K rows are rotated ("rotate-half" pairs
// (j, j + d/2), angle pos * theta^(-2j/d)) and written to their page slots, V rows are copied bit for
// bit, and, if asked, the step's query rows are rotated in place by the same positions.
//
// Angles and the rotation are evaluated in fp64 and rounded once (fp64 -> fp32 -> bf16, nearest even):
// positions reach 10^5, where an fp32 angle would already be off by several thousandths of a radian.
// The kernel moves a few MB; the arithmetic is not worth economising.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>

#include <algorithm>

#include "asynclm.h"
#include "common.cuh"
#include "kernels.h"
#include "plan_internal.h"

namespace asynclm {

namespace {

__device__ __forceinline__ float bf16_to_f32(unsigned short b) { return __uint_as_float((unsigned)b << 16); }
__device__ __forceinline__ unsigned short f64_to_bf16(double x) {
    const __nv_bfloat16 h = __float2bfloat16_rn(__double2float_rn(x));
    return *reinterpret_cast<const unsigned short*>(&h);
}

// One thread rotates the two 16-byte vectors (values 8v .. 8v+7 and their partners d/2 further) of one
// row of one head.  rows: K rows [T][Hkv][d] (then written to the pool) and, optionally, Q rows
// [T][Hq][d] (rewritten in place); V rows are copied by the threads of the K rows.
__global__ void __launch_bounds__(256)
kv_append_rope_kernel(DevPlan p, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                      uint4* __restrict__ pool, uint4* __restrict__ q, double log2_theta) {
    const int d = p.head_dim, half_vecs = d / 16;                 // vectors in half a row
    const int heads_k = p.num_kv_heads, heads_q = q != nullptr ? p.num_q_heads : 0;
    const int64_t per_token = (int64_t)(heads_k + heads_q) * half_vecs;
    const int64_t total = (int64_t)p.total_q * per_token;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(idx / per_token);
        int rest = (int)(idx % per_token);
        const int v = rest % half_vecs;
        const int h = rest / half_vecs;                              // kv heads first, then query heads
        const int b = __ldg(p.row_seq + r);
        const int pos = __ldg(p.kv_len_before + b) + r - __ldg(p.q_indptr + b);
        const bool is_k = h < heads_k;
        const uint4* src = is_k ? k_new + ((size_t)r * heads_k + h) * (2 * half_vecs)
                                : q + ((size_t)r * heads_q + (h - heads_k)) * (2 * half_vecs);
        const uint4 lo = src[v], hi = src[v + half_vecs];
        const unsigned short* xl = reinterpret_cast<const unsigned short*>(&lo);
        const unsigned short* xh = reinterpret_cast<const unsigned short*>(&hi);
        uint4 olo, ohi;
        unsigned short* yl = reinterpret_cast<unsigned short*>(&olo);
        unsigned short* yh = reinterpret_cast<unsigned short*>(&ohi);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = 8 * v + k;
            double s, c;
            sincos((double)pos * exp2(-2.0 * (double)j / (double)d * log2_theta), &s, &c);
            const double a = (double)bf16_to_f32(xl[k]), bb = (double)bf16_to_f32(xh[k]);
            yl[k] = f64_to_bf16(a * c - bb * s);
            yh[k] = f64_to_bf16(bb * c + a * s);
        }
        if (is_k) {
            const int64_t ps = __ldg(p.row_slot + r);
            if (!page_ok(ps / kPage, p.num_pages, p.status, kStatusBadPageAppend)) continue;
            const size_t dst = pool_row_offset(ps / kPage, 0, h, (int)(ps % kPage), heads_k, d) / 8;
            pool[dst + v] = olo;
            pool[dst + v + half_vecs] = ohi;
            // the V row of the same (token, head): a bit copy
            const uint4* vs = v_new + ((size_t)r * heads_k + h) * (2 * half_vecs);
            const size_t vd = pool_row_offset(ps / kPage, 1, h, (int)(ps % kPage), heads_k, d) / 8;
            pool[vd + v] = vs[v];
            pool[vd + v + half_vecs] = vs[v + half_vecs];
        } else {
            uint4* dst = q + ((size_t)r * heads_q + (h - heads_k)) * (2 * half_vecs);
            dst[v] = olo;
            dst[v + half_vecs] = ohi;
        }
    }
}

}  // namespace

}  // namespace asynclm

extern "C" int asynclm_kv_append_rope(const asynclm_plan_t* plan, const void* k_new, const void* v_new, void* kv_pool,
                                      void* q_inout, double rope_theta, void* stream) {
    using namespace asynclm;
    if (!plan || plan->magic != kPlanMagic || plan->host_only || !(rope_theta > 1.0)) return ASYNCLM_ERR_INVALID_ARG;
    if (plan->dev.total_q == 0) return ASYNCLM_OK;
    if (!k_new || !v_new || !kv_pool || (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)kv_pool | (uintptr_t)q_inout) & 15) != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    if (int rc = check_plan_device(plan->device)) return rc;
    const DevPlan& p = plan->dev;
    const int64_t total = (int64_t)p.total_q * (p.num_kv_heads + (q_inout ? p.num_q_heads : 0)) * (p.head_dim / 16);
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, 148 * 8);
    kv_append_rope_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(p, (const uint4*)k_new, (const uint4*)v_new,
                                                                    (uint4*)kv_pool, (uint4*)q_inout, log2(rope_theta));
    return cuda_status(cudaGetLastError());
}
