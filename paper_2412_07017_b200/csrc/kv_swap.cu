// Trap handler data path (paper Section 5.4): while a sequence waits for an interrupt its KV cache can
// be swapped to host memory and brought back later, possibly into other pages.  The swapped form of a
// sequence is its pages in logical order, one contiguous image [n_pages][2][Hkv][16][d].
//
// Swap-out gathers the pages into a contiguous device staging buffer with one kernel and then moves
// the image to (pinned) host memory with ONE asynchronous copy, so that PCIe sees a single long
// transfer instead of one per page; swap-in is the mirror image.  The keep / swap / recompute rule of
// the same section is evaluated on the host by asynclm_trap_decide.
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "asynclm.h"
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

// A page is one contiguous run of `vpp` 16-byte vectors in the pool; page j of the image is page ids[j]
// of the pool.  Four vectors in flight per thread; consecutive threads take consecutive vectors.
template <bool TO_POOL>
__global__ void __launch_bounds__(256)
page_copy_kernel(uint4* __restrict__ pool, uint4* __restrict__ image, const int32_t* __restrict__ ids,
                 int64_t total, int vpp) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < total; i0 += 4 * stride) {
        uint4 v[4];
        int64_t at[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = i0 + u * stride;
            at[u] = -1;
            if (i < total) {
                at[u] = (int64_t)__ldg(ids + i / vpp) * vpp + i % vpp;
                v[u] = TO_POOL ? ldg_nc_v4(image + i) : ldg_nc_v4(pool + at[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = i0 + u * stride;
            if (at[u] >= 0) {
                if (TO_POOL) pool[at[u]] = v[u];
                else image[i] = v[u];
            }
        }
    }
}

static size_t page_bytes(const asynclm_shape* s) {
    return (size_t)2 * s->num_kv_heads * s->page_size * s->head_dim * 2;
}

static int check_swap_args(const asynclm_shape* s, const int32_t* ids, int32_t n, const void* pool, const void* staging,
                           const void* host_image, bool distinct) {
    if (!s || s->num_kv_heads <= 0 || s->page_size <= 0 || s->head_dim <= 0 || s->head_dim % 8 != 0 || n < 0)
        return ASYNCLM_ERR_INVALID_ARG;
    if (n == 0) return ASYNCLM_OK;
    if (!ids || !pool || !staging || !host_image || (((uintptr_t)pool | (uintptr_t)staging | (uintptr_t)host_image) & 15) != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    for (int32_t j = 0; j < n; ++j)
        if (ids[j] < 0 || ids[j] >= s->num_pages) return ASYNCLM_ERR_PAGE_TABLE;
    if (distinct) {
        std::vector<int32_t> sorted(ids, ids + n);
        std::sort(sorted.begin(), sorted.end());
        if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return ASYNCLM_ERR_PAGE_TABLE;
    }
    return ASYNCLM_OK;
}

static int grid_for(int64_t total) {
    const int64_t blocks = (total + 4 * 256 - 1) / (4 * 256);
    return (int)std::min<int64_t>(std::max<int64_t>(blocks, 1), 148 * 8);
}

}  // namespace asynclm

using namespace asynclm;

extern "C" size_t asynclm_kv_swap_staging_bytes(const asynclm_shape* shape, int32_t n_pages) {
    if (!shape || n_pages < 0) return 0;
    return (size_t)n_pages * page_bytes(shape) + (((size_t)n_pages * 4 + 255) / 256) * 256;
}

extern "C" int asynclm_kv_swap_out(const asynclm_shape* shape, const int32_t* page_ids, int32_t n_pages,
                                   const void* kv_pool, void* staging, void* host_image, void* stream) {
    if (int rc = check_swap_args(shape, page_ids, n_pages, kv_pool, staging, host_image, false)) return rc;
    if (n_pages == 0) return ASYNCLM_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t bytes = (size_t)n_pages * page_bytes(shape);
    int32_t* ids_dev = reinterpret_cast<int32_t*>((char*)staging + bytes);
    if (int rc = cuda_status(cudaMemcpyAsync(ids_dev, page_ids, (size_t)n_pages * 4, cudaMemcpyHostToDevice, s))) return rc;
    const int vpp = (int)(page_bytes(shape) / 16);
    const int64_t total = (int64_t)n_pages * vpp;
    page_copy_kernel<false><<<grid_for(total), 256, 0, s>>>((uint4*)const_cast<void*>(kv_pool), (uint4*)staging, ids_dev, total, vpp);
    if (int rc = cuda_status(cudaGetLastError())) return rc;
    return cuda_status(cudaMemcpyAsync(host_image, staging, bytes, cudaMemcpyDeviceToHost, s));
}

extern "C" int asynclm_kv_swap_in(const asynclm_shape* shape, const int32_t* page_ids, int32_t n_pages,
                                  void* kv_pool, void* staging, const void* host_image, void* stream) {
    if (int rc = check_swap_args(shape, page_ids, n_pages, kv_pool, staging, host_image, true)) return rc;
    if (n_pages == 0) return ASYNCLM_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t bytes = (size_t)n_pages * page_bytes(shape);
    int32_t* ids_dev = reinterpret_cast<int32_t*>((char*)staging + bytes);
    if (int rc = cuda_status(cudaMemcpyAsync(ids_dev, page_ids, (size_t)n_pages * 4, cudaMemcpyHostToDevice, s))) return rc;
    if (int rc = cuda_status(cudaMemcpyAsync(staging, host_image, bytes, cudaMemcpyHostToDevice, s))) return rc;
    const int vpp = (int)(page_bytes(shape) / 16);
    const int64_t total = (int64_t)n_pages * vpp;
    page_copy_kernel<true><<<grid_for(total), 256, 0, s>>>((uint4*)kv_pool, (uint4*)staging, ids_dev, total, vpp);
    return cuda_status(cudaGetLastError());
}

extern "C" int asynclm_trap_decide(const asynclm_trap_model* model, int32_t context_tokens, double wait_us,
                                   int32_t* decision, double* swap_us, double* recompute_us) {
    if (!model || !decision || context_tokens < 0 || !(wait_us >= 0.0)) return ASYNCLM_ERR_INVALID_ARG;
    const double n = (double)context_tokens;
    const double s = model->swap_fixed_us + model->swap_us_per_token * n;
    const double r = model->recompute_fixed_us + model->recompute_us_per_token * n + model->recompute_us_per_token2 * n * n;
    if (swap_us) *swap_us = s;
    if (recompute_us) *recompute_us = r;
    if (s > wait_us && r > wait_us) *decision = ASYNCLM_TRAP_KEEP;
    else *decision = r < s ? ASYNCLM_TRAP_RECOMPUTE : ASYNCLM_TRAP_SWAP;
    return ASYNCLM_OK;
}
