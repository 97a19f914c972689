// Split-KV merge: combine the per-chunk (normalised output, log-sum-exp) pairs of one row,
//     LSE = log sum_c exp(LSE_c),   O = sum_c exp(LSE_c - LSE) O_c,
// in chunk order, so the result does not depend on which CTA produced which chunk.
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

template <int D>
__global__ void __launch_bounds__(128)
lse_merge_kernel(DevPlan p, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    constexpr int EPL = D / 32;   // output elements per lane
    const int lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    const Unit u = p.units[p.split_units[blockIdx.x]];
    const int G = p.group;
    // one warp per (token, head) pair of the unit; blockIdx.y tiles the unit's pairs
    const int pair = blockIdx.y * nwarps + (threadIdx.x >> 5);
    if (pair < u.ntok * G) {
        const int t = pair / G, g = pair % G;
        float mx = -INFINITY;
        for (int c = 0; c < u.n_chunks; ++c) {
            const size_t prow = (size_t)u.partial_base + (size_t)c * u.ntok + t;
            mx = fmaxf(mx, p.partial_lse[prow * G + g]);
        }
        float acc[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
        float wsum = 0.f;
        for (int c = 0; c < u.n_chunks; ++c) {
            const size_t prow = (size_t)u.partial_base + (size_t)c * u.ntok + t;
            const float l2 = p.partial_lse[prow * G + g];
            if (l2 == -INFINITY) continue;     // chunk with no visible key for this row
            const float w = fast_exp2(l2 - mx);
            wsum += w;
            const float* src = p.partial_o + (prow * G + g) * D + lane * EPL;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = fmaf(w, src[e], acc[e]);
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
    if (p.num_split_units == 0) return cudaSuccess;
    // a unit has at most 128 (token, head) pairs (a tensor-core tile); CUDA-core units have G
    const int max_pairs = p.num_items_tensor > 0 ? 128 : p.group;
    const dim3 grid(p.num_split_units, (max_pairs + 3) / 4);
    if (p.head_dim == 128)
        lse_merge_kernel<128><<<grid, 128, 0, stream>>>(p, (__nv_bfloat16*)out, lse);
    else
        lse_merge_kernel<64><<<grid, 128, 0, stream>>>(p, (__nv_bfloat16*)out, lse);
    return cudaGetLastError();
}

}  // namespace asynclm
