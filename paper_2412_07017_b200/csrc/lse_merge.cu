// Split-KV merge: combine the per-chunk (normalised output, log-sum-exp) pairs of one row,
//     LSE = log sum_c exp(LSE_c),   O = sum_c exp(LSE_c - LSE) O_c.
// One warp per (token, head) row that was split, four rows per CTA (the planner lists the row
// blocks); chunks are added in chunk order, so the result does not depend on which CTA produced
// which chunk or on scheduling.
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

template <int D>
__global__ void __launch_bounds__(128)
lse_merge_kernel(DevPlan p, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    constexpr int EPL = D / 32;   // output elements per lane
    const int lane = threadIdx.x & 31;
    const int G = p.group;
    // the plan was uploaded before the attention kernel started: read it while that kernel drains
    const int entry = p.merge_blocks[blockIdx.x];
    const Unit u = p.units[entry >> 6];
    pdl_wait();     // the partial results are complete and visible from here on
    const int pair = (entry & 63) * 4 + (threadIdx.x >> 5);
    if (pair >= u.ntok * G) return;
    const int t = pair / G, g = pair % G;
    const int n = u.n_chunks;
    const size_t prow0 = (size_t)u.partial_base + t;       // chunk c -> prow0 + c * ntok
    // maximum of the chunks' log-sum-exps, chunks spread over the lanes
    float mx = -INFINITY;
    for (int c = lane; c < n; c += 32)
        mx = fmaxf(mx, p.partial_lse[(prow0 + (size_t)c * u.ntok) * G + g]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    float wsum = 0.f;
    // weighted sum in chunk order, eight loads in flight at a time
    for (int c0 = 0; c0 < n; c0 += 8) {
        float w[8];
        float v[8][EPL];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int c = c0 + k;
            w[k] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) v[k][e] = 0.f;
            if (c < n) {
                const size_t prow = prow0 + (size_t)c * u.ntok;
                const float l2 = p.partial_lse[prow * G + g];
                w[k] = l2 == -INFINITY ? 0.f : fast_exp2(l2 - mx);   // -inf: no visible key in that chunk
                const float* src = p.partial_o + (prow * G + g) * D + lane * EPL;
#pragma unroll
                for (int e = 0; e < EPL; ++e) v[k][e] = src[e];
            }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            wsum += w[k];
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = w[k] != 0.f ? fmaf(w[k], v[k][e], acc[e]) : acc[e];
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

cudaError_t launch_lse_merge(const DevPlan& p, void* out, float* lse, cudaStream_t stream) {
    if (p.num_merge_blocks == 0) return cudaSuccess;
    // Programmatic serialization: the attention kernels let their dependents start as soon as all of
    // their CTAs are running, so this grid's launch and plan reads overlap the attention tail.
    if (p.head_dim == 128)
        return launch_pdl(lse_merge_kernel<128>, dim3(p.num_merge_blocks), dim3(128), 0, stream, p,
                          (__nv_bfloat16*)out, lse);
    return launch_pdl(lse_merge_kernel<64>, dim3(p.num_merge_blocks), dim3(128), 0, stream, p,
                      (__nv_bfloat16*)out, lse);
}

}  // namespace asynclm
