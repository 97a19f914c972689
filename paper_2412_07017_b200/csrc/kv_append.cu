// Interrupt append: scatter the new K/V rows of a step into their page slots, bit for bit.
//
// An interrupt block goes to the end of the sequence's context (paper Section 3.2); a decode token
// is the span of length one.  Row i of sequence b lands at position ctx_b + i, i.e. in physical
// page page_indices[page_indptr[b] + pos / 16], slot pos % 16.
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

// One 16-byte vector per thread; consecutive threads cover one 2*d-byte row, so both the read and
// the write of a row are single coalesced segments.
__global__ void __launch_bounds__(256)
kv_append_kernel(DevPlan p, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                 uint4* __restrict__ pool) {
    pdl_trigger();   // the attention kernel may start its prologue; it waits for this grid before reading the pool
    const int vpr = p.head_dim / 8;                       // 16-byte vectors per row
    const int64_t total = (int64_t)p.total_q * p.num_kv_heads * 2 * vpr;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int vec = (int)(idx % vpr);
        int64_t rest = idx / vpr;
        const int h = (int)(rest % p.num_kv_heads);
        rest /= p.num_kv_heads;
        const int which = (int)(rest & 1);
        const int r = (int)(rest >> 1);
        // the planner resolved the row's page and slot (position ctx_b + i through the page table), so
        // the slot and the source row are fetched side by side instead of through four dependent loads
        const int64_t ps = __ldg(p.row_slot + r);
        const uint4 val = ldg_nc_v4((which ? v_new : k_new) + ((size_t)r * p.num_kv_heads + h) * vpr + vec);
        if (!page_ok(ps / kPage, p.num_pages, p.status, kStatusBadPageAppend)) continue;
        const size_t dst = pool_row_offset(ps / kPage, which, h, (int)(ps % kPage), p.num_kv_heads, p.head_dim) / 8 + vec;
        pool[dst] = val;
    }
}

cudaError_t launch_kv_append(const DevPlan& p, const void* k_new, const void* v_new, void* kv_pool,
                             cudaStream_t stream) {
    if (p.total_q == 0) return cudaSuccess;
    const int64_t total = (int64_t)p.total_q * p.num_kv_heads * 2 * (p.head_dim / 8);
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    kv_append_kernel<<<blocks, 256, 0, stream>>>(p, (const uint4*)k_new, (const uint4*)v_new,
                                                 (uint4*)kv_pool);
    return cudaGetLastError();
}

}  // namespace asynclm
