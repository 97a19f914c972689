// The attention kernels' entry points and launchers.
//
// Three kernels are built from two bodies (attn_append_tc.cuh: tensor-core span tiles,
// attn_decode.cuh: CUDA-core decode rows):
//   attn_fused_kernel      a persistent CTA first runs its tensor-core items, then its CUDA-core items
//                          (a CTA without span tiles skips the tensor-memory set-up altogether).
//                          One launch instead of two: the fixed cost of a launch (about 10 us of
//                          start-up and tail per kernel at 148 CTAs) is paid once, and a CTA that is
//                          done with its span tiles early moves on to decode rows at once.
//   attn_append_tc_kernel  steps that have span tiles only
//   attn_decode_kernel     steps without span tiles, and head_dim 64
// All are launched with programmatic stream serialization and wait for the kernel in front of them
// (normally the KV append) right before they first touch the pool.
#include <atomic>

#include "attn_append_tc.cuh"
#include "attn_decode.cuh"

namespace asynclm {

namespace {

constexpr int kMaxSmem = 232448;

__device__ __forceinline__ uint8_t* aligned_smem(uint8_t* raw) {
    return (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
}

template <int D, int G, bool APPEND>
__global__ void __launch_bounds__(dec::kThreads, 1)
attn_decode_kernel(DevPlan p, const __grid_constant__ CUtensorMap kv_map, const __nv_bfloat16* __restrict__ q,
                   __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int S, AppendSrc app) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();      // the split-KV merge behind this kernel may start its prologue
    if (threadIdx.x == 0) { trace_mark(0); trace_set(1, 0); trace_set(5, 0); trace_set(6, 0); trace_set(7, 0); }
    dec::decode_body<D, G, APPEND>(p, &kv_map, q, out, lse, S, aligned_smem(smem_raw), app);
}

template <int G, bool APPEND>
__global__ void __launch_bounds__(tc::kThreads, 1)
attn_append_tc_kernel(DevPlan p, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* pool,
                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse, AppendSrc app) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();      // the kernel behind this one may start its prologue; it waits for this grid to complete
    if (threadIdx.x == 0) {
        trace_mark(0);
        for (int s = 8; s < 16; ++s) trace_set(s, 0);
    }
    tc::tc_body<G, APPEND>(p, q, pool, out, lse, aligned_smem(smem_raw), app);
    if (threadIdx.x == 0) trace_mark(1);
}

template <int G, bool APPEND>
__global__ void __launch_bounds__(tc::kThreads, 1)
attn_fused_kernel(DevPlan p, const __grid_constant__ CUtensorMap kv_map, const __nv_bfloat16* __restrict__ q,
                  const __nv_bfloat16* pool, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                  int S, AppendSrc app) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = aligned_smem(smem_raw);
    pdl_trigger();      // the split-KV merge behind this kernel may start its prologue
    if (threadIdx.x == 0) { trace_mark(0); trace_set(1, 0); trace_set(5, 0); trace_set(6, 0); trace_set(7, 0); }
    const int32_t* head = p.cta_heads + (size_t)blockIdx.x * kHeadWords;
    // bring the whole header and the tensor map close now: the decode phase of a CTA that starts with
    // span tiles finds them in L2 when it gets there
    if (threadIdx.x < 3) asm volatile("prefetch.global.L2 [%0];" ::"l"(head + 32 * threadIdx.x));
    if (threadIdx.x == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&kv_map));
    if (head[0] == head[1]) {
        // no span tiles for this CTA: straight to its decode rows, without the tensor-memory set-up
        dec::decode_body<tc::kD, G, APPEND>(p, &kv_map, q, out, lse, S, smem, app);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 8; s < 16; ++s) trace_set(s, 0);
    }
    tc::tc_body<G, APPEND>(p, q, pool, out, lse, smem, app);
    if (threadIdx.x == 0) trace_mark(1);
    if (head[2] == head[3] && p.queue_count == 0) return;      // nothing left for the warp body
    __syncthreads();      // tensor memory released, shared memory free for the second phase
    dec::decode_body<tc::kD, G, APPEND>(p, &kv_map, q, out, lse, S, smem, app);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The pool as a 5-D tensor (64 values, 16 slots, d / 64 row halves, Hkv, pages x K|V) with a box of
// one page's K and V blocks of one kv head, landed with the 128-byte swizzle (see dec::tma_page_kv).
// The driver entry point is looked up once per process.
cudaError_t make_kv_map(const DevPlan& p, const void* pool, CUtensorMap* map) {
    static std::atomic<EncodeTiledFn> encode_fn{nullptr};
    EncodeTiledFn encode = encode_fn.load(std::memory_order_acquire);
    if (encode == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
        encode = (EncodeTiledFn)sym;
        encode_fn.store(encode, std::memory_order_release);
    }
    const cuuint64_t d = (cuuint64_t)p.head_dim, hkv = (cuuint64_t)p.num_kv_heads;
    if (p.num_pages <= 0 || p.num_pages > 0x3fffffff) return cudaErrorInvalidValue;
    const cuuint64_t dims[5] = {64, kPage, d / 64, hkv, 2 * (cuuint64_t)p.num_pages};
    const cuuint64_t strides[4] = {d * 2, 128, kPage * d * 2, hkv * kPage * d * 2};
    const cuuint32_t box[5] = {64, kPage, (cuuint32_t)(d / 64), 1, 2};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of once per launch.
// The kernel is a template VALUE: kernels of one signature share a pointer type, and a flag per type
// would let the first of them stand for all.
template <auto kernel>
cudaError_t allow_smem(size_t bytes) {
    static std::atomic<unsigned long long> done{0};      // one per kernel instantiation; bit = device (first 64)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = dev < 64 ? 1ull << dev : 0ull;
    if (bit != 0 && (done.load(std::memory_order_acquire) & bit) != 0) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && bit != 0) done.fetch_or(bit, std::memory_order_release);
    return e;
}

// The tensor map of a pool depends on its address and shape only: the last few are kept per thread.
cudaError_t cached_kv_map(const DevPlan& p, const void* pool, CUtensorMap* map) {
    struct Entry { const void* pool; int64_t pages; int hkv, d; CUtensorMap map; };
    constexpr int kEntries = 8;
    thread_local Entry cache[kEntries] = {};
    thread_local int next = 0;
    for (int i = 0; i < kEntries; ++i)
        if (cache[i].pool == pool && cache[i].pages == p.num_pages && cache[i].hkv == p.num_kv_heads && cache[i].d == p.head_dim) {
            *map = cache[i].map;
            return cudaSuccess;
        }
    const cudaError_t e = make_kv_map(p, pool, map);
    if (e == cudaSuccess) {
        cache[next] = Entry{pool, p.num_pages, p.num_kv_heads, p.head_dim, *map};
        next = (next + 1) % kEntries;
    }
    return e;
}

template <int D>
int decode_stages() {
    int S = 6;
    while (S > 2 && dec::smem_bytes<D>(S) > (size_t)kMaxSmem) --S;
    return S;
}

template <int D, int G, bool APPEND>
cudaError_t launch_decode(const DevPlan& p, const void* q, const void* pool, void* out, float* lse,
                          cudaStream_t stream, AppendSrc app) {
    const int S = decode_stages<D>();
    const size_t smem = dec::smem_bytes<D>(S);
    cudaError_t e = allow_smem<attn_decode_kernel<D, G, APPEND>>(smem);
    if (e != cudaSuccess) return e;
    CUtensorMap map;
    e = cached_kv_map(p, pool, &map);
    if (e != cudaSuccess) return e;
    return launch_pdl(attn_decode_kernel<D, G, APPEND>, dim3(p.num_ctas_cuda), dim3(dec::kThreads), smem, stream, p, map,
                      (const __nv_bfloat16*)q, (__nv_bfloat16*)out, lse, S, app);
}

template <int G, bool APPEND>
cudaError_t launch_tensor(const DevPlan& p, const void* q, const void* pool, void* out, float* lse,
                          cudaStream_t stream, AppendSrc app) {
    cudaError_t e = allow_smem<attn_append_tc_kernel<G, APPEND>>(tc::kSmemBytes);
    if (e != cudaSuccess) return e;
    return launch_pdl(attn_append_tc_kernel<G, APPEND>, dim3(p.num_ctas_tensor), dim3(tc::kThreads), tc::kSmemBytes, stream,
                      p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)pool, (__nv_bfloat16*)out, lse, app);
}

template <int G, bool APPEND>
cudaError_t launch_fused(const DevPlan& p, const void* q, const void* pool, void* out, float* lse,
                         cudaStream_t stream, AppendSrc app) {
    const int S = decode_stages<tc::kD>();
    const size_t smem = dec::smem_bytes<tc::kD>(S) > tc::kSmemBytes ? dec::smem_bytes<tc::kD>(S) : tc::kSmemBytes;
    cudaError_t e = allow_smem<attn_fused_kernel<G, APPEND>>(smem);
    if (e != cudaSuccess) return e;
    CUtensorMap map;
    e = cached_kv_map(p, pool, &map);
    if (e != cudaSuccess) return e;
    return launch_pdl(attn_fused_kernel<G, APPEND>, dim3(p.num_ctas_cuda), dim3(tc::kThreads), smem, stream, p, map,
                      (const __nv_bfloat16*)q, (const __nv_bfloat16*)pool, (__nv_bfloat16*)out, lse, S, app);
}

template <int D, bool APPEND>
cudaError_t launch_decode_d(const DevPlan& p, const void* q, const void* pool, void* out, float* lse,
                            cudaStream_t stream, AppendSrc app) {
    switch (p.group) {
        case 1: return launch_decode<D, 1, APPEND>(p, q, pool, out, lse, stream, app);
        case 2: return launch_decode<D, 2, APPEND>(p, q, pool, out, lse, stream, app);
        case 4: return launch_decode<D, 4, APPEND>(p, q, pool, out, lse, stream, app);
        case 8: return launch_decode<D, 8, APPEND>(p, q, pool, out, lse, stream, app);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool tensor_path_compiled(int head_dim) { return head_dim == tc::kD; }

namespace {

template <bool APPEND>
cudaError_t launch_attention_impl(const DevPlan& p, const void* q, const void* kv_pool, void* out, float* lse,
                                  cudaStream_t stream, AppendSrc app) {
    const bool has_tensor = p.num_items_tensor > 0, has_cuda = p.num_items_cuda > 0;
    if (has_tensor && p.head_dim != tc::kD) return cudaErrorInvalidValue;
    if (has_tensor && has_cuda && p.num_ctas_tensor == p.num_ctas_cuda) {
        switch (p.group) {
            case 1: return launch_fused<1, APPEND>(p, q, kv_pool, out, lse, stream, app);
            case 2: return launch_fused<2, APPEND>(p, q, kv_pool, out, lse, stream, app);
            case 4: return launch_fused<4, APPEND>(p, q, kv_pool, out, lse, stream, app);
            case 8: return launch_fused<8, APPEND>(p, q, kv_pool, out, lse, stream, app);
            default: return cudaErrorInvalidValue;
        }
    }
    if (has_tensor) {
        cudaError_t e;
        switch (p.group) {
            case 1: e = launch_tensor<1, APPEND>(p, q, kv_pool, out, lse, stream, app); break;
            case 2: e = launch_tensor<2, APPEND>(p, q, kv_pool, out, lse, stream, app); break;
            case 4: e = launch_tensor<4, APPEND>(p, q, kv_pool, out, lse, stream, app); break;
            case 8: e = launch_tensor<8, APPEND>(p, q, kv_pool, out, lse, stream, app); break;
            default: e = cudaErrorInvalidValue;
        }
        if (e != cudaSuccess) return e;
    }
    if (has_cuda) {
        // a decode kernel behind a tensor kernel would have to wait for it to finish (pdl_wait), which
        // is what stream order gives anyway
        if (p.head_dim == 128) return launch_decode_d<128, APPEND>(p, q, kv_pool, out, lse, stream, app);
        if (p.head_dim == 64) return launch_decode_d<64, APPEND>(p, q, kv_pool, out, lse, stream, app);
        return cudaErrorInvalidValue;
    }
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_attention(const DevPlan& p, const void* q, const void* kv_pool, void* out, float* lse,
                             cudaStream_t stream, AppendSrc app) {
    return app.k_new != nullptr ? launch_attention_impl<true>(p, q, kv_pool, out, lse, stream, app)
                                : launch_attention_impl<false>(p, q, kv_pool, out, lse, stream, app);
}

}  // namespace asynclm

#ifdef ASYNCLM_TRACE
// Debug builds only: copies the per-CTA time stamps of the last attention launch to the host
// (synchronises the device).  out: [1024][8] unsigned 64-bit.
extern "C" int asynclm_trace_read(unsigned long long* out) {
    return cudaMemcpyFromSymbol(out, asynclm::g_trace, sizeof(asynclm::g_trace)) == cudaSuccess ? 0 : -5;
}
// The event log of the first CTAs: out [4][11][512] unsigned 64-bit (cycle << 8 | event); clears it.
extern "C" int asynclm_trace_events_read(unsigned long long* out) {
    if (cudaMemcpyFromSymbol(out, asynclm::g_events, sizeof(asynclm::g_events)) != cudaSuccess) return -5;
    void* dev = nullptr;
    if (cudaGetSymbolAddress(&dev, asynclm::g_events) != cudaSuccess) return -5;
    return cudaMemset(dev, 0, sizeof(asynclm::g_events)) == cudaSuccess ? 0 : -5;
}
#endif