// Measurement aid: how fast can this GPU read the K/V blocks of a step at all?
//
// The attention kernels read, for every (sequence, kv head), the K block and the V block (16 slots x
// head_dim bf16 each, contiguous) of every page of the sequence, pages scattered over the pool.  This
// kernel reads exactly such a list of blocks with plain 16-byte loads and no arithmetic beyond an XOR
// that keeps the loads alive: persistent CTAs of 1024 threads, a contiguous share of the list each,
// eight loads in flight per thread.  Its rate is the ceiling the attention kernels are compared with beside
// the copy bandwidth (a copy also writes).  It holds none of the method's arithmetic.
#include <cuda_runtime.h>
#include <stdint.h>

#include "asynclm.h"
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

// k_offsets[i]: byte offset of a K block in the pool; its V block lies v_delta bytes further; a block has
// `vecs` 16-byte vectors (2 * vecs divides 1024).  The CTA's 1024 threads cover 1024 / (2 vecs) pairs at
// a time, one vector each, and keep eight such rows in flight: 128 KB per SM.
__global__ void __launch_bounds__(1024, 1)
read_ceiling_kernel(const uint8_t* __restrict__ pool, const int64_t* __restrict__ k_offsets, int64_t n,
                    int64_t v_delta, int vecs, unsigned* __restrict__ sink) {
    constexpr int U = 8;
    const int per_row = 1024 / (2 * vecs);                 // pairs per row of loads
    const int sub = threadIdx.x / (2 * vecs), t = threadIdx.x % (2 * vecs);
    const int64_t within = t < vecs ? (int64_t)t * 16 : v_delta + (int64_t)(t - vecs) * 16;
    unsigned acc = 0;
    // every CTA takes one contiguous share of the list, as an attention CTA takes the consecutive pages
    // of a sequence
    const int64_t share = (n + gridDim.x - 1) / gridDim.x;
    const int64_t begin = share * blockIdx.x, end = begin + share < n ? begin + share : n;
    for (int64_t i = begin; i < end; i += (int64_t)per_row * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t idx = i + (int64_t)u * per_row + sub;
            v[u] = idx < end ? ldg_nc_v4(pool + k_offsets[idx] + within) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    if (acc == 0x9e3779b9u) sink[0] = acc;      // practically never; keeps the loads
}

}  // namespace asynclm

extern "C" int asynclm_read_ceiling(const void* kv_pool, const int64_t* k_block_offsets, int64_t n_blocks,
                                    int64_t v_delta_bytes, int32_t block_bytes, void* sink, void* stream) {
    using namespace asynclm;
    if (!kv_pool || !sink || n_blocks < 0 || (n_blocks > 0 && !k_block_offsets) || block_bytes < 16 ||
        512 % (block_bytes / 16) != 0 || block_bytes % 16 != 0 || (((uintptr_t)kv_pool | (uintptr_t)v_delta_bytes) & 15) != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    if (n_blocks == 0) return ASYNCLM_OK;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_status(e);
    read_ceiling_kernel<<<sms, 1024, 0, (cudaStream_t)stream>>>((const uint8_t*)kv_pool, k_block_offsets, n_blocks,
                                                                v_delta_bytes, block_bytes / 16, (unsigned*)sink);
    return cuda_status(cudaGetLastError());
}
