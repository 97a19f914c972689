// Small device helpers shared by the kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan_types.h"

namespace asynclm {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Two bf16 values packed in a 32-bit word -> two floats (exact).
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Two floats -> packed bf16x2, round to nearest even (lo in the low half).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while the kernel before it in the stream is still running; pdl_wait() blocks until that
// kernel has completed and its writes are visible, pdl_trigger() lets the next kernel start early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with the programmatic-serialization attribute (see pdl_wait / pdl_trigger).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Per-CTA time stamps for performance work: compiled in only with -DASYNCLM_TRACE (see build.py),
// read back with asynclm_trace_read().  Slot meanings are the callers'.
#ifdef ASYNCLM_TRACE
constexpr int kTraceSlots = 16, kTraceCtas = 1024;
static __device__ unsigned long long g_trace[kTraceCtas][kTraceSlots];      // one copy per translation unit
__device__ __forceinline__ void trace_mark(int slot) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    if (blockIdx.x < kTraceCtas) g_trace[blockIdx.x][slot] = t;
}
__device__ __forceinline__ void trace_add(int slot, unsigned long long v) {
    if (blockIdx.x < kTraceCtas) g_trace[blockIdx.x][slot] += v;
}
__device__ __forceinline__ void trace_set(int slot, unsigned long long v) {
    if (blockIdx.x < kTraceCtas) g_trace[blockIdx.x][slot] = v;
}
__device__ __forceinline__ long long trace_clock() { return clock64(); }
// Event log of the first kEventCtas CTAs: (SM cycle counter << 8 | event id) in the order a role
// (one thread) records them; `n` is the role's own count.
constexpr int kEventCtas = 4, kEventRoles = 11, kEventsPerRole = 512;
static __device__ unsigned long long g_events[kEventCtas][kEventRoles][kEventsPerRole];
__device__ __forceinline__ void trace_event(int role, int& n, int id) {
    if (blockIdx.x < kEventCtas && n < kEventsPerRole)
        g_events[blockIdx.x][role][n++] = ((unsigned long long)clock64() << 8) | (unsigned)id;
}
#else
__device__ __forceinline__ void trace_event(int, int&, int) {}
__device__ __forceinline__ long long trace_clock() { return 0; }
__device__ __forceinline__ void trace_mark(int) {}
__device__ __forceinline__ void trace_add(int, unsigned long long) {}
__device__ __forceinline__ void trace_set(int, unsigned long long) {}
#endif

// Checked build (-DASYNCLM_DEBUG, see build.py): every page id a kernel is about to turn into an address is
// compared with the pool's size first; a bad one puts `code` into the status word (the first one wins)
// and the caller leaves the access out.  The ordinary build relies on the planner, which validates every
// id on the host, and compiles the check away.
#ifdef ASYNCLM_DEBUG
__device__ __forceinline__ bool page_ok(int64_t page, int64_t num_pages, int32_t* status, int code) {
    if (page >= 0 && page < num_pages) return true;
    atomicCAS(status, 0, code);
    return false;
}
#else
__device__ __forceinline__ bool page_ok(int64_t, int64_t, int32_t*, int) { return true; }
#endif
constexpr int kStatusBadPageAppend = 41, kStatusBadPageSpan = 42, kStatusBadPageWarp = 43, kStatusBadPageStep = 44;

// Element offset of the first value of (page, K|V, kv head, slot) in the pool.
__device__ __forceinline__ size_t pool_row_offset(int64_t page, int which, int kv_head, int slot,
                                                  int num_kv_heads, int head_dim) {
    return ((((size_t)page * 2 + (size_t)which) * (size_t)num_kv_heads + (size_t)kv_head) * kPage +
            (size_t)slot) * (size_t)head_dim;
}

// Interrupt append inside an attention kernel (paper Section 3.2: the block goes to the end of the
// context): one warp copies, bit for bit, the new K/V rows of one kv head that an item is about to
// read, positions [max(kv0, ctx), kv_end) of its sequence, from k_new / v_new into their page slots.
// Every item does this for the rows it reads itself, so no CTA ever waits for another; items that
// read the same rows write the same bytes.  `w`: the item's Work record.
__device__ __forceinline__ void append_rows_of_item(const DevPlan& p, const AppendSrc& app, const Work& w, int lane) {
    const int ctx = w.kv_limit0 - 1 - (w.q_row0 - w.q_seq0);
    const int lo = max(w.kv0, ctx);
    const int vpr = p.head_dim / 8;                       // 16-byte vectors per row
    const int total = (w.kv_end - lo) * 2 * vpr;
    const uint4* k_new = reinterpret_cast<const uint4*>(app.k_new);
    const uint4* v_new = reinterpret_cast<const uint4*>(app.v_new);
    uint4* pool = reinterpret_cast<uint4*>(app.pool);
    // sixteen vectors per lane are requested together, then stored: the copy is a chain of round trips
    // to memory otherwise
    constexpr int kBatch = 16;
    for (int base = lane; base < total; base += 32 * kBatch) {
        uint4 val[kBatch];
        size_t dst[kBatch];
        bool ok[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = base + 32 * j;
            if (i < total) {
                const int pos = lo + i / (2 * vpr), r = i % (2 * vpr);
                const int which = r / vpr, vec = r % vpr;
                int64_t page = __ldg(p.page_indices + w.page0 + (pos - w.kv0) / kPage);
                ok[j] = page_ok(page, p.num_pages, p.status, kStatusBadPageStep);
                if (!ok[j]) page = 0;
                val[j] = ldg_nc_v4((which ? v_new : k_new) + ((size_t)(w.q_seq0 + pos - ctx) * p.num_kv_heads + w.kv_head) * vpr + vec);
                dst[j] = pool_row_offset(page, which, w.kv_head, pos % kPage, p.num_kv_heads, p.head_dim) / 8 + vec;
            }
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j)
            if (base + 32 * j < total && ok[j]) pool[dst[j]] = val[j];
    }
}

}  // namespace asynclm
