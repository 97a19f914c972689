// Split-KV merge: combine the per-chunk (normalised output, log-sum-exp) pairs of one row,
//     LSE = log sum_c exp(LSE_c),   O = sum_c exp(LSE_c - LSE) O_c.
// One warp per (token, head) row that was split, 4 rows per CTA (the planner lists the row
// blocks); chunks are added in chunk order, so the result does not depend on which CTA produced
// which chunk or on scheduling.
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

// A block takes 4 (token, head) rows of one split unit, one per warp.  (Measured: blocks of 512
// threads with two rows per warp were slower; late blocks of a dependent grid are dispatched slowly,
// so small blocks that fit beside each other early do better.)
constexpr int kMergeThreads = 128;
constexpr int kMergeRows = 4;

template <int D>
__global__ void __launch_bounds__(kMergeThreads)
lse_merge_kernel(DevPlan p, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    constexpr int EPL = D / 32;   // output elements per lane
    const int lane = threadIdx.x & 31;
    const int G = p.group;
    // the plan was uploaded before the attention kernel started: read it while that kernel drains
    const int entry = p.merge_blocks[blockIdx.x];
    const Unit u = p.units[entry >> 6];
    const int pair = (entry & 63) * kMergeRows + (threadIdx.x >> 5);
    if (pair < u.ntok * G) {
        // Touch the row's partial results ahead of the wait: the data is not final yet, but the address
        // translations are, and a first touch from this SM costs more than the L2 hit that follows.
        const size_t prow = (size_t)u.partial_base + pair / G;
        for (int c = lane; c < u.n_chunks; c += 32) {
            const size_t r = (prow + (size_t)c * u.ntok) * G + pair % G;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.partial_lse + r));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p.partial_o + r * D));
        }
    }
    pdl_wait();     // the partial results are complete and visible from here on
  {
    if (pair >= u.ntok * G) return;
    const int t = pair / G, g = pair % G;
    const int n = u.n_chunks;
    const size_t prow0 = (size_t)u.partial_base + t;       // chunk c -> prow0 + c * ntok
    // Up to eight chunks per pass: their log-sum-exps and their outputs are requested together (one
    // round trip to L2, where the attention kernel has just left them), then weighted in chunk order
    // against a running maximum.
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    float mx = -INFINITY, wsum = 0.f;
    for (int c0 = 0; c0 < n; c0 += 8) {
        float l2[8];
        float v[8][EPL];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int c = c0 + k;
            l2[k] = -INFINITY;
#pragma unroll
            for (int e = 0; e < EPL; ++e) v[k][e] = 0.f;
            if (c < n) {
                const size_t prow = prow0 + (size_t)c * u.ntok;
                l2[k] = p.partial_lse[prow * G + g];
                const float* src = p.partial_o + (prow * G + g) * D + lane * EPL;
                if constexpr (EPL == 4) {
                    const float4 x = *reinterpret_cast<const float4*>(src);
                    v[k][0] = x.x; v[k][1] = x.y; v[k][2] = x.z; v[k][3] = x.w;
                } else {
                    const float2 x = *reinterpret_cast<const float2*>(src);
                    v[k][0] = x.x; v[k][1] = x.y;
                }
            }
        }
        float pm = mx;
#pragma unroll
        for (int k = 0; k < 8; ++k) pm = fmaxf(pm, l2[k]);
        const float rescale = pm == -INFINITY ? 1.f : fast_exp2(mx - pm);      // first pass: exp2(-inf) = 0
        mx = pm;
        wsum *= rescale;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= rescale;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float w = l2[k] == -INFINITY ? 0.f : fast_exp2(l2[k] - mx);   // -inf: no visible key in that chunk
            wsum += w;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = w != 0.f ? fmaf(w, v[k][e], acc[e]) : acc[e];
        }
    }
    const float inv = 1.f / wsum;
    const size_t row = (size_t)u.q_row0 + t;
    const size_t hq = (size_t)u.kv_head * G + g;
    __nv_bfloat16* dst = out + (row * p.num_q_heads + hq) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; e += 2)
        *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
    if (lse != nullptr && lane == 0)
        lse[row * p.num_q_heads + hq] = (mx + log2f(wsum)) * kLn2;
  }
}

cudaError_t launch_lse_merge(const DevPlan& p, void* out, float* lse, cudaStream_t stream) {
    if (p.num_merge_blocks == 0) return cudaSuccess;
    // Programmatic serialization: the attention kernels let their dependents start as soon as all of
    // their CTAs are running, so this grid's launch and plan reads overlap the attention tail.
    if (p.head_dim == 128)
        return launch_pdl(lse_merge_kernel<128>, dim3(p.num_merge_blocks), dim3(kMergeThreads), 0, stream, p,
                          (__nv_bfloat16*)out, lse);
    return launch_pdl(lse_merge_kernel<64>, dim3(p.num_merge_blocks), dim3(kMergeThreads), 0, stream, p,
                      (__nv_bfloat16*)out, lse);
}

}  // namespace asynclm
