// Tensor-core attention for interrupt spans (tcgen05 MMA, accumulators and P in tensor memory).
//
// An interrupt span is a block of new tokens appended to one sequence (paper Section 3.2); in the
// next decoding step (Section 5.3) every token of the span attends to the whole cached context and
// causally to the span itself.  With G query heads per kv head, a span of q tokens gives G*q query
// rows against the same K/V, which is a dense contraction: rows are packed 128 to a tile
// (row r = token r / G, head r % G) and S = Q K^T and O += P V run on the tensor cores.
//
// A work item covers up to 256 query rows (two row tiles) of one (sequence, kv head) and a range of
// keys.  One persistent CTA per SM, twelve working warps:
//   warps 0-3, 4-7  two softmax groups, one thread per query row of a tile.  Each group owns one S
//                   accumulator (128 fp32 columns of tensor memory) and one O accumulator.
//                     * items with more than 128 rows ("dual"): group b owns row tile b and both
//                       groups consume every KV tile, so K and V are fetched once for 256 rows;
//                     * items with at most 128 rows: the groups take alternate KV tiles of the one
//                       row tile and their (max, sum, O) states are merged in the epilogue like two
//                       KV splits.
//                   The softmax runs in place: a thread reads its row of S 64 columns at a time and
//                   writes P as packed bf16 pairs over the columns it has already read; P V then
//                   takes its A operand from tensor memory.  The reference maximum only moves when
//                   a score exceeds it by 2^8; then O, the running sum and the half of P already
//                   written are rescaled.  With one softmax warp per scheduler the stage is bound
//                   by issue slots and dependent latency, so the arithmetic around the exponentials
//                   is packed two values to an instruction and reductions run in independent chains.
//                   At the end of an item the rows go out through the group's (now idle) Q tile in
//                   shared memory, so that every global store writes whole 128-byte lines.
//   warps 8, 10     producers of K tiles and of V tiles: 16-byte cp.async copies (fully coalesced,
//                   two 256-byte rows per warp instruction) that write the 128-byte-swizzled operand
//                   layout and complete on the slot's mbarrier.  K and V share one ring of five
//                   32 KiB slots, filled in the order the tensor core consumes them
//                   (K0 K1 V0 K2 V1 K3 ...): a V tile is needed one softmax later than the K tile
//                   of the same keys, and a shared ring lets whichever is due use the free slots.
//   warp 9          one thread issues all MMAs, a group at a time (P V of its tile, then Q K^T of its
//                   next tile), so that the groups' softmaxes alternate instead of colliding on the
//                   exponential unit.  The warp owns the tensor-memory allocation.
//   warp 11         idle, except when the kernel appends the step's new K/V rows itself
//                   (asynclm_step): then it runs ahead of the producers and copies, item by item, the
//                   new rows the item reads into their page slots; the producers wait for an item's
//                   rows before they fetch its first tile.
// All hand-offs are mbarriers with bounded waits; a wait that runs out sets the plan's status word
// and a CTA-wide abort flag, every role falls through to the common exit, and the tensor memory is
// released there.
#pragma once
#include <climits>

#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace tc {

constexpr int kThreads = 384;
constexpr int kProducerWarpK = 8, kMmaWarp = 9, kProducerWarpV = 10, kAppendWarp = 11;
constexpr int kD = 128;
constexpr int kTile = 128;                       // keys per K/V ring slot and query rows per row tile
constexpr int kSub = 64;                         // keys the softmax handles at a time (half an S tile)
// Pairs (of the 16 of a quarter) whose exponentials are evaluated by polynomial instead of ex2.approx.
#ifndef ASYNCLM_POLY_MASK
#define ASYNCLM_POLY_MASK 0x4924u
#endif
constexpr uint32_t kPolyMask = ASYNCLM_POLY_MASK;
constexpr int kRing = 5;                         // K/V ring slots
constexpr uint32_t kHalfBytes = 128 * 128;       // one 64-value half of a 128-row tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;  // 32 KiB
constexpr float kRescaleThreshold = 8.f;
constexpr long long kWaitCycles = 2000000000ll;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;                           // Q[0], Q[1]
constexpr uint32_t kOffRing = kOffQ + 2 * kTileBytes;
constexpr uint32_t kOffBar = kOffRing + kRing * kTileBytes;
// S, P V and P hand-offs exist per group b: index 2 * b
enum Bar { kQFull = 0, kStats, kOFree, kPFull0, kPvDone0 = kPFull0 + 4, kSFull0 = kPvDone0 + 4,
           kRingFull0 = kSFull0 + 4, kRingEmpty0 = kRingFull0 + kRing, kMmaDrain = kRingEmpty0 + kRing,
           kNumBars };
constexpr uint32_t kOffTmemPtr = kOffBar + 8 * kNumBars;
constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
constexpr uint32_t kOffAppended = kOffAbort + 8;      // items of this CTA whose new K/V rows are in the pool
constexpr uint32_t kSmemBytes = kOffAppended + 8 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");

// tensor memory columns
constexpr uint32_t kColS = 0;      // S[0], S[1]: 128 columns each; P[b] overlays the first 64 of S[b]
constexpr uint32_t kColO = 256;    // O[0], O[1]: 128 columns each
constexpr uint32_t kTmemCols = 512;

// Ring position of the K tile and of the V tile of the CTA's g-th KV tile: K0 K1 V0 K2 V1 K3 ...
__device__ __forceinline__ int ring_pos_k(int g) { return g == 0 ? 0 : 2 * g - 1; }
__device__ __forceinline__ int ring_pos_v(int g) { return 2 * g + 2; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        __nanosleep(32);      // leave the issue slots to the warps that have work
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicCAS(status, 0, code);
            return false;
        }
    }
    return true;
}
// The same wait without the back-off, for the one thread that issues the MMAs: what it waits for is on
// the critical path of both softmax groups.
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* status, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            atomicCAS(status, 0, code);
            return false;
        }
    }
    return true;
}
// The same wait with a warp-uniform verdict, for code that goes on to warp-collective instructions.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* status, int code) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status, code));
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// Arrive on the mbarrier once all cp.async copies issued so far by this thread have landed.
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n; b_mn = 1 when B is stored with N
// contiguous (the V tile), 0 when K is contiguous.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\tselp.u32 %0, 1, 0, e;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define TC_R32(r) \
    "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), \
    "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), \
    "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), \
    "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
#define TC_W32(r) \
    "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), \
    "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), \
    "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), \
    "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])

// This warp's 32 rows x 32 consecutive fp32 columns of tensor memory -> one row per thread.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : TC_R32(r) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
        ::TC_W32(r), "r"(taddr) : "memory");
}
// Waits for this thread's tensor-memory loads; the loaded registers pass through the statement so that
// no use of them can be scheduled in front of it.
__device__ __forceinline__ void tmem_wait_ld_dep(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 16 consecutive 32-bit columns of this warp's 32 rows.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t& a, uint32_t& b) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(a), "=r"(b) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st2(uint32_t taddr, uint32_t a, uint32_t b) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%2], {%0,%1};" ::"r"(a), "r"(b), "r"(taddr) : "memory");
}
// D (+)= A B with A taken from tensor memory: row i of A is lane i, its 16 bf16 values of one K step
// are 8 consecutive 32-bit columns (two values per column, the lower index in the low half).
__device__ __forceinline__ void mma_f16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}

// 2^x for two finite values on the FMA pipe: n = round(x) through the 1.5 * 2^23 trick, a cubic for
// 2^(x - n) on [-1/2, 1/2] (relative error 7.5e-5, below the bf16 rounding of P), n added to the
// exponent field.  x is clamped at -125 so that the exponent cannot wrap.
__device__ __forceinline__ float2 poly_exp2(float2 x) {
    const float kMagic = 12582912.f;
    const float2 xc = make_float2(fmaxf(x.x, -125.f), fmaxf(x.y, -125.f));
    const float2 t = __fadd2_rn(xc, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), xc);
    float2 r = __ffma2_rn(f, make_float2(0.0551716685f, 0.0551716685f), make_float2(0.2426111251f, 0.2426111251f));
    r = __ffma2_rn(r, f, make_float2(0.6932609677f, 0.6932609677f));
    r = __ffma2_rn(r, f, make_float2(0.9999280572f, 0.9999280572f));
    return make_float2(__int_as_float(__float_as_int(r.x) + (__float_as_int(t.x) << 23)),
                       __int_as_float(__float_as_int(r.y) + (__float_as_int(t.y) << 23)));
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// One work item as the kernel sees it (kv_end == 0: no item).
struct TItem {
    int kv0, kv_end, q_row0, ntok, kv_limit0, kv_head, partial_row0, page0;
};

// `rec`: a Work record (the planner's array, or the copy of a CTA's first item in its header).
__device__ __forceinline__ TItem load_titem(const Work* rec, bool valid) {
    TItem r{0, 0, 0, 0, 0, 0, -1, 0};
    if (valid) {
        const int4* src = reinterpret_cast<const int4*>(rec);
        const int4 a = __ldg(src), b = __ldg(src + 1);
        r.kv0 = a.x; r.kv_end = a.y; r.q_row0 = a.z; r.ntok = a.w;
        r.kv_limit0 = b.x; r.kv_head = b.y; r.partial_row0 = b.z; r.page0 = b.w;
    }
    return r;
}

// The whole kernel body, called by all twelve warps with `smem` 1024-byte aligned.
template <int G, bool APPEND>
__device__ __forceinline__ void tc_body(const DevPlan& p, const __nv_bfloat16* __restrict__ q,
                                        const __nv_bfloat16* pool,
                                        __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                        uint8_t* smem, const AppendSrc& app) {
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_ptr = (volatile uint32_t*)(smem + kOffTmemPtr);
    volatile int* abort_flag = (volatile int*)(smem + kOffAbort);
    volatile int* appended = (volatile int*)(smem + kOffAppended);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int Hq = p.num_q_heads, Hkv = p.num_kv_heads;
    // The plan was uploaded before the kernel in front of this one started, so it may be read before
    // pdl_wait(); everything else (pool, q, outputs) is touched only after it.
    const int32_t* head = p.cta_heads + (size_t)blockIdx.x * kHeadWords;
    const int i0 = head[0], i1 = head[1];
    const Work* head_work = reinterpret_cast<const Work*>(head + kHeadWorkTensor);      // = p.works[i0]

    if (threadIdx.x == 0) {
        mbar_init(bar(kQFull), 256);
        mbar_init(bar(kStats), 256);
        mbar_init(bar(kOFree), 256);
        for (int b = 0; b < 4; ++b) {
            mbar_init(bar(kPFull0 + b), 4);      // one arrival per warp of the group
            mbar_init(bar(kPvDone0 + b), 1);
            mbar_init(bar(kSFull0 + b), 1);
        }
        for (int s = 0; s < kRing; ++s) { mbar_init(bar(kRingFull0 + s), 32); mbar_init(bar(kRingEmpty0 + s), 1); }
        mbar_init(bar(kMmaDrain), 1);
        *abort_flag = 0;
        *appended = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(sbase + kOffTmemPtr), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_ptr;

    if (warp >= 8) {
      if (warp == kProducerWarpK || warp == kProducerWarpV) {
        // ------------------------------------------------------------------ producer warps
        const int which = warp == kProducerWarpV ? 1 : 0;       // 0: K tiles, 1: V tiles
        const uint32_t ring = sbase + kOffRing;
        auto load_pages = [&](const TItem& it, int first_page) {
            const int npg = (it.kv_end - it.kv0 + kPage - 1) / kPage;
            const int idx = first_page + lane;
            return idx < npg ? __ldg(p.page_indices + it.page0 + idx) : 0;
        };
        constexpr int kPagesPerTile = kTile / kPage;          // 8
        constexpr int kGroupTiles = 32 / kPagesPerTile;       // 4
        bool ok = true;
        int n = 0;                                             // KV tiles issued so far (all items)
        int last_pos = -1;
        int ev = 0;      // time-stamp build: event log position (lane 0 of a producer)
        TItem cur = load_titem(head_work, i0 < i1), nxt = load_titem(p.works + i0 + 1, i0 + 1 < i1);
        int pages_cur = head[kHeadPagesTensor + lane];      // the first item's first 32 page ids (0 beyond its end)
        pdl_wait();
        for (int ii = i0; cur.kv_end > 0 && ok; ++ii) {
            const TItem after = load_titem(p.works + ii + 2, ii + 2 < i1);
            const int ntiles = (cur.kv_end - cur.kv0 + kTile - 1) / kTile;
            // APPEND: the first key position of the item that this step appends; tiles up to it are
            // fetched at once, the others only when the append warp has put the rows in the pool
            int first_new = INT_MAX;
            if constexpr (APPEND) {
                const int q_seq0 = ii == i0 ? head_work->q_seq0 : __ldg(&p.works[ii].q_seq0);
                first_new = cur.kv_limit0 - 1 - (cur.q_row0 - q_seq0);
            }
            bool appended_seen = false;
            for (int t0 = 0; t0 < ntiles && ok; t0 += kGroupTiles) {
                int pages_nxt = 0;
                const int t1 = min(t0 + kGroupTiles, ntiles);
                for (int t = t0; t < t1 && ok; ++t, ++n) {
                    const int rows = min(kTile, cur.kv_end - (cur.kv0 + t * kTile));
                    const int npages = (rows + kPage - 1) / kPage;
                    if constexpr (APPEND) {
                        if (!appended_seen && cur.kv0 + t * kTile + rows > first_new) {
                            const long long t_wait = clock64();
                            while (*appended <= ii - i0 && ok) {
                                __nanosleep(64);
                                if (*abort_flag) ok = false;
                                else if (clock64() - t_wait > kWaitCycles) {
                                    *abort_flag = 1;
                                    atomicCAS(p.status, 0, 13);
                                    ok = false;
                                }
                            }
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                            __threadfence();
                            appended_seen = true;
                        }
                    }
                    const int pos = which ? ring_pos_v(n) : ring_pos_k(n);
                    const int s = pos % kRing;
                    if (lane == 0) trace_event(9 + which, ev, 40);
                    ok = mbar_wait_warp(bar(kRingEmpty0 + s), ((uint32_t)(pos / kRing) & 1u) ^ 1u, abort_flag, p.status, 11 + which);
                    if (!ok) break;
                    if (lane == 0) trace_event(9 + which, ev, 42);
                    last_pos = pos;
                    // lane -> 16-byte chunk c of row 2*rr + (lane >> 4) of each page: a warp instruction
                    // moves two whole 256-byte rows
                    const int c = lane & 15;
                    const uint32_t dst_half = ring + s * kTileBytes + (uint32_t)(c >> 3) * kHalfBytes;
                    for (int pg = 0; pg < npages; ++pg) {
                        int64_t page = __shfl_sync(0xffffffffu, pages_cur, (t - t0) * kPagesPerTile + pg);
                        const bool page_good = page_ok(page, p.num_pages, p.status, kStatusBadPageSpan);      // checked build only
                        if (!page_good) page = 0;      // the tile gets zeros in its place
                        const uint8_t* src_page = reinterpret_cast<const uint8_t*>(
                            pool + pool_row_offset(page, which, cur.kv_head, 0, Hkv, kD));
#pragma unroll
                        for (int rr = 0; rr < kPage / 2; ++rr) {
                            const int slot = rr * 2 + (lane >> 4);
                            const int row = pg * kPage + slot;
                            cp_async16(dst_half + (uint32_t)row * 128u + (uint32_t)(((c & 7) ^ (row & 7)) << 4),
                                       src_page + slot * (kD * 2) + c * 16, (row < rows && page_good) ? 16u : 0u);
                        }
                    }
#ifdef ASYNCLM_DEBUG
                    // checked build: a test may ask for one hand-off to be left out, to see a bounded wait run out
                    if (!(which == 0 && blockIdx.x == 0 && p.debug_stall_tile == n + 1))
#endif
                    cp_async_arrive(bar(kRingFull0 + s));
                    if (lane == 0) trace_event(9 + which, ev, 44);
                    // page ids of the next group of tiles (or of the next item), requested only after this
                    // group's first tile is on its way: the next item's descriptor may still be in flight
                    if (t == t0) {
                        if (t0 + kGroupTiles < ntiles) pages_nxt = load_pages(cur, (t0 + kGroupTiles) * kPagesPerTile);
                        else if (nxt.kv_end > 0) pages_nxt = load_pages(nxt, 0);
                    }
                }
                pages_cur = pages_nxt;
            }
            cur = nxt;
            nxt = after;
        }
        if (!ok && last_pos >= 0) {
            // aborted: let the loads already issued land before shared memory goes away
            asm volatile("cp.async.wait_all;" ::: "memory");
        }
      } else if (warp == kAppendWarp) {
        // ------------------------------------------------------------------ append warp (asynclm_step only)
        if constexpr (APPEND) {
            pdl_wait();
            for (int ii = i0; ii < i1; ++ii) {
                const Work rec = ii == i0 ? *head_work : p.works[ii];
                append_rows_of_item(p, app, rec, lane);
                __threadfence();      // the rows are visible device-wide before the count moves
                __syncwarp();
                if (lane == 0) *appended = ii - i0 + 1;
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        // One warp, running convergently, issues every MMA of the CTA through an elected lane (operands then
        // stay in uniform registers: under a lane-0 branch each MMA took the lone thread 85-110 cycles to
        // issue, against 64 cycles on the tensor core), in an order that lets the two softmax groups work
        // in turns: after the P V of a group's tile it issues the Q K^T of the same group's next tile
        // at once (MMAs of one thread execute in issue order, so the new S may overwrite the P that the
        // P V in front of it reads), then it turns to the other group.  While the tensor core works
        // for one group, the other group's softmax has the exponential unit to itself.
        // Q K^T is issued 128 keys wide (8 instructions per tile and group, 64 cycles each on the tensor
        // core): narrower instructions cost nearly as much to issue.
        {
            bool ok = true;
            int gt = 0;               // KV tiles before this item (all items): ring position
            int cnt0 = 0, cnt1 = 0;   // tiles whose P V has been issued, per group: phase of the P hand-off
            int item_no = 0;
            const uint32_t idesc_pv = instr_desc(128, 1);
            TItem it_next = load_titem(head_work, i0 < i1);
            const long long t_loop = trace_clock();
            long long tr_p = 0, tr_kv = 0, tr_item = 0, tr_qk = 0, tr_pv = 0;      // time-stamp build: cycles waiting for P, for K/V, for an item's Q and O
            int ev = 0;                                                            // time-stamp build: event log position
            for (int ii = i0; ii < i1 && ok; ++ii, ++item_no) {
                const TItem it = it_next;
                it_next = load_titem(p.works + ii + 1, ii + 1 < i1);      // in flight while this item runs
                const int ntiles = (it.kv_end - it.kv0 + kTile - 1) / kTile;
                const bool dual = it.ntok * G > kTile;
                const long long t_item = trace_clock();
                if (lane == 0) trace_event(0, ev, 1);
                ok = mbar_wait_spin(bar(kQFull), (uint32_t)item_no & 1u, abort_flag, p.status, 22);
                // S and O of the previous item are in use until its epilogue is over
                if (ok && item_no > 0) ok = mbar_wait_spin(bar(kOFree), (uint32_t)(item_no - 1) & 1u, abort_flag, p.status, 27);
                tr_item += trace_clock() - t_item;
                if (lane == 0) trace_event(0, ev, 2);
                if (ok) tc_fence_after();
                auto tile_pages = [&](int j) { return (min(kTile, it.kv_end - (it.kv0 + j * kTile)) + kPage - 1) / kPage; };
                // Hand-offs the MMAs of a turn wait for.  K/V tiles first (they are normally there already),
                // P last, so that nothing stands between its arrival and the first MMA.
                auto wait_k = [&](int j) {
                    const int pos = ring_pos_k(gt + j), s = pos % kRing;
                    const long long tw = trace_clock();
                    ok = ok && mbar_wait_spin(bar(kRingFull0 + s), (uint32_t)(pos / kRing) & 1u, abort_flag, p.status, 21);
                    tr_kv += trace_clock() - tw;
                };
                auto wait_v = [&](int j) {
                    const int pos = ring_pos_v(gt + j), s = pos % kRing;
                    const long long tw = trace_clock();
                    ok = ok && mbar_wait_spin(bar(kRingFull0 + s), (uint32_t)(pos / kRing) & 1u, abort_flag, p.status, 24);
                    tr_kv += trace_clock() - tw;
                };
                auto wait_p = [&](int b) {
                    const long long tw = trace_clock();
                    ok = ok && mbar_wait_spin(bar(kPFull0 + 2 * b), (uint32_t)(b ? cnt1 : cnt0) & 1u, abort_flag, p.status, 26);
                    tr_p += trace_clock() - tw;
                };
                // S[b] <- Q[qt] K_j^T, then one commit: it tells group b that S[b] is complete and, because MMAs
                // complete in issue order, that every MMA in front of it is done as well (the group releases
                // the ring slots on that knowledge: a second commit per batch costs the tensor pipe ~90 cycles)
                auto emit_qk = [&](int j, int b) {
                    const long long ti = trace_clock();
                    const int s = ring_pos_k(gt + j) % kRing;
                    const uint32_t idesc = instr_desc(16u * (uint32_t)tile_pages(j), 0);
                    const uint32_t d = tmem + kColS + 128u * (uint32_t)b;
                    const uint64_t qd = smem_desc(sbase + kOffQ + (dual ? (uint32_t)b * kTileBytes : 0u), 16, 1024);
                    const uint64_t kd = smem_desc(sbase + kOffRing + s * kTileBytes, 16, 1024);
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        // the address field counts 16-byte units and cannot carry out of its 14 bits here
                        const uint64_t off = (uint64_t)(((uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u) >> 4);
                        if (elect_one()) mma_f16(d, qd + off, kd + off, idesc, ks > 0);
                    }
                    if (elect_one()) mma_commit(bar(kSFull0 + 2 * b));
                    tr_qk += trace_clock() - ti;
                    if (lane == 0) trace_event(0, ev, 14 + b);
                };
                // O[b] (+)= P[b] V_j with P[b] in tensor memory; fresh: first P V of the item into O[b];
                // last: the group's last tile of the item, the only one whose completion is signalled by itself
                auto emit_pv = [&](int j, int b, bool fresh, bool last) {
                    const long long ti = trace_clock();
                    const int s = ring_pos_v(gt + j) % kRing;
                    const int npg = tile_pages(j);
                    const uint32_t pcol = tmem + kColS + 128u * (uint32_t)b;
                    const uint64_t vd = smem_desc(sbase + kOffRing + s * kTileBytes, kHalfBytes, 1024);
                    const uint32_t ocol = tmem + kColO + 128u * (uint32_t)b;
                    if (npg == kTile / kPage) {
#pragma unroll
                        for (int ks = 0; ks < kTile / kPage; ++ks)
                            if (elect_one()) mma_f16_ta(ocol, pcol + 8u * (uint32_t)ks, vd + (uint64_t)(ks * 128), idesc_pv, (!fresh || ks > 0) ? 1u : 0u);
                    } else {
                        for (int ks = 0; ks < npg; ++ks)
                            if (elect_one()) mma_f16_ta(ocol, pcol + 8u * (uint32_t)ks, vd + (uint64_t)(ks * 128), idesc_pv, (!fresh || ks > 0) ? 1u : 0u);
                    }
                    if (last && elect_one()) mma_commit(bar(kPvDone0 + 2 * b));
                    if (b) ++cnt1; else ++cnt0;
                    tr_pv += trace_clock() - ti;
                    if (lane == 0) trace_event(0, ev, 26 + b);
                };
                auto first_qk = [&](int j, int b) {
                    wait_k(j);
                    if (!ok) return;
                    tc_fence_after();
                    emit_qk(j, b);
                };
                // One turn of group b: the P V of its tile j and at once the Q K^T of its next tile jn (-1: none),
                // sixteen MMAs issued back to back once everything they read is there.
                auto turn = [&](int j, int b, bool fresh, int jn) {
                    if (lane == 0) trace_event(0, ev, 20 + b);
                    wait_v(j);
                    if (jn >= 0) wait_k(jn);
                    wait_p(b);
                    if (lane == 0) trace_event(0, ev, 22 + b);
                    if (!ok) return;
                    tc_fence_after();
                    emit_pv(j, b, fresh, jn < 0);
                    if (jn >= 0) emit_qk(jn, b);
                };
                if (dual) {
                    // both groups on every tile: group b owns row tile b
                    first_qk(0, 0);
                    if (ok) first_qk(0, 1);
                    for (int j = 0; j < ntiles && ok; ++j)
                        for (int b = 0; b < 2 && ok; ++b) turn(j, b, j == 0, j + 1 < ntiles ? j + 1 : -1);
                } else {
                    // one row tile: the groups take alternate KV tiles
                    first_qk(0, 0);
                    if (ok && ntiles > 1) first_qk(1, 1);
                    for (int j = 0; j < ntiles && ok; ++j) turn(j, j & 1, j < 2, j + 2 < ntiles ? j + 2 : -1);
                }
                gt += ntiles;
            }
            if (lane == 0) {
                trace_set(8, tr_p);
                trace_set(9, tr_kv);
                trace_set(10, trace_clock() - t_loop);
                trace_set(14, tr_item);
                trace_set(2, tr_qk);
                trace_set(3, tr_pv);
            }
            // make sure nothing is still running on the tensor core before tensor memory is released
            if (elect_one()) mma_commit(bar(kMmaDrain));
            const long long t0 = clock64();
            while (!mbar_try_wait(bar(kMmaDrain), 0) && clock64() - t0 < kWaitCycles) {}
        }
        __syncwarp();
      }
    } else {
        // ------------------------------------------------------------------ softmax / epilogue groups
        const int b = warp >> 2;                   // softmax group
        const int m = threadIdx.x & 127;           // row of the group's tile = tensor-memory lane
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_addr = lane_addr + kColS + 128u * (uint32_t)b;      // + 64 * buffer
        const uint32_t o_addr = lane_addr + kColO + 128u * (uint32_t)b;
        const float qscale = p.sm_scale * kLog2e;
        const float2 qscale2 = make_float2(qscale, qscale);
        int cnt = 0;         // tiles this group has processed before this item
        int gt = 0;          // KV tiles of the CTA before this item (both groups): ring position
        int pv_cnt = 0;      // items so far in which this group had tiles: phase of its "last P V done" barrier
        int item_no = 0;
        bool ok = true;
        long long tr_wait = 0, tr_work = 0, tr_tiles = 0;      // time-stamp build: cycles waiting for S, cycles from S to P, tiles
        int ev = 0;                                            // time-stamp build: event log position (lane 0 of each warp)
        // This thread's share of an item's Q.  Dual items: the whole row 128 b + m (16 chunks of 16
        // bytes) into Q[b]; otherwise value half b of row m (8 chunks) into Q[0].  The next item's Q is
        // fetched at the end of the current item's KV loop, ahead of the epilogue.
        auto load_q = [&](const TItem& x, uint4 (&w)[16]) {
            const bool dual = x.ntok * G > kTile;
            const int r = dual ? 128 * b + m : m;
            const bool valid = x.kv_end > 0 && r / G < x.ntok;
            const uint4* src = reinterpret_cast<const uint4*>(
                q + ((size_t)(x.q_row0 + r / G) * Hq + (size_t)x.kv_head * G + r % G) * kD) + (dual ? 0 : 8 * b);
#pragma unroll
            for (int c = 0; c < 8; ++c) w[c] = valid ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int c = 8; c < 16; ++c) w[c] = (valid && dual) ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
        };
        TItem it_next = load_titem(head_work, i0 < i1);
        uint4 q_next[16];
        pdl_wait();
        load_q(it_next, q_next);
        for (int ii = i0; ii < i1 && ok; ++ii, ++item_no) {
            const TItem it = it_next;
            const int ntiles = (it.kv_end - it.kv0 + kTile - 1) / kTile;
            const bool dual = it.ntok * G > kTile;
            const int r = dual ? 128 * b + m : m;      // query row of the item
            const int t = r / G, g = r % G;
            const bool row_valid = t < it.ntok;
            // ---- stage Q with the 128-byte swizzle the MMA descriptor expects (the previous item's
            // epilogue used the Q tiles as its output staging area: wait until every warp is through)
            if (item_no > 0) {
                ok = mbar_wait_warp(bar(kOFree), (uint32_t)(item_no - 1) & 1u, abort_flag, p.status, 36);
                if (!ok) break;
            }
            if (dual) {
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    *reinterpret_cast<uint4*>(smem + kOffQ + b * kTileBytes + (c >> 3) * kHalfBytes + m * 128 +
                                              (((c & 7) ^ (m & 7)) << 4)) = q_next[c];
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4*>(smem + kOffQ + b * kHalfBytes + m * 128 + ((c ^ (m & 7)) << 4)) = q_next[c];
            }
            fence_async_smem();
            mbar_arrive(bar(kQFull));
            if (lane == 0) trace_event(1 + warp, ev, 37);
            it_next = load_titem(p.works + ii + 1, ii + 1 < i1);
            const int lim_row = row_valid ? min(it.kv_limit0 + t, it.kv_end) : 0;   // keys [0, lim_row) visible
            float m_ref = -INFINITY;                     // reference maximum (log2 domain)
            float2 l2 = make_float2(0.f, 0.f), l2b = make_float2(0.f, 0.f);      // running sum of P, four partial sums
            int mine = 0;                                // tiles of this group so far in this item
            for (int j = dual ? 0 : b; j < ntiles && ok; j += dual ? 1 : 2, ++mine) {
                const int npg = (min(kTile, it.kv_end - (it.kv0 + j * kTile)) + kPage - 1) / kPage;
                // S[b] complete; it was issued after the P V of this group's previous tile finished, so
                // O[b] is at rest as well
                const long long tw = trace_clock();
                if (lane == 0) trace_event(1 + warp, ev, 30);
                ok = __all_sync(0xffffffffu, mbar_wait_spin(bar(kSFull0 + 2 * b), (uint32_t)(cnt + mine) & 1u, abort_flag, p.status, 31));
                const long long ts = trace_clock();
                if (lane == 0) trace_event(1 + warp, ev, 31);
                tr_wait += ts - tw;
                ++tr_tiles;
                if (!ok) break;
                tc_fence_after();
                // S[b] of tile j complete means every MMA issued before it is complete.  The group that is
                // last to use a ring slot gives it back to the producers: the K tile of j now, and the V tile
                // of the group's previous tile (its P V was issued in front of this Q K^T).
                if (m == 0 && (!dual || b == 1)) {
                    mbar_arrive(bar(kRingEmpty0 + ring_pos_k(gt + j) % kRing));
                    if (mine > 0) mbar_arrive(bar(kRingEmpty0 + ring_pos_v(gt + j - (dual ? 1 : 2)) % kRing));
                }
                // the tile is handled in two halves of 64 keys (register budget)
                for (int h = 0; h * 4 < npg; ++h) {
                    const int base = it.kv0 + j * kTile + h * kSub;
                    const int vis = max(0, min(kSub, lim_row - base));      // visible columns of this row
                    const uint32_t sb = s_addr + 64u * (uint32_t)h;
                    uint32_t rr[64];
                    tmem_ld32(sb, *reinterpret_cast<uint32_t(*)[32]>(&rr[0]));
                    tmem_ld32(sb + 32u, *reinterpret_cast<uint32_t(*)[32]>(&rr[32]));
                    tmem_wait_ld();
                    // x = S * scale - m_ref (log2 domain), two values per instruction
                    const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
                    const float2 nm2 = make_float2(-m_use, -m_use);
                    float2 x[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        x[e] = __ffma2_rn(make_float2(__uint_as_float(rr[2 * e]), __uint_as_float(rr[2 * e + 1])), qscale2, nm2);
                    if (!__all_sync(0xffffffffu, vis == kSub)) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            if (2 * e >= vis) x[e].x = -INFINITY;
                            if (2 * e + 1 >= vis) x[e].y = -INFINITY;
                        }
                    }
                    // row maximum of the half: four independent chains of 3-input maxima (a lone warp per
                    // scheduler cannot hide one long dependent chain)
                    auto xv = [&](int k) { return (k & 1) ? x[k >> 1].y : x[k >> 1].x; };
                    float cm[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) cm[c] = fmax3(xv(16 * c), xv(16 * c + 1), xv(16 * c + 2));
#pragma unroll
                    for (int k = 3; k < 15; k += 2) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) cm[c] = fmax3(cm[c], xv(16 * c + k), xv(16 * c + k + 1));
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) cm[c] = fmaxf(cm[c], xv(16 * c + 15));
                    const float cmax = fmax3(fmaxf(cm[0], cm[1]), cm[2], cm[3]);
                    // x is relative to m_ref (to 0 while the row has no reference yet: then any visible key sets it)
                    if (__any_sync(0xffffffffu, cmax > (m_ref == -INFINITY ? -INFINITY : kRescaleThreshold))) {
                        // Move the reference maximum (rare after the first tile): rescale the running sum, the
                        // half of P already written for this tile and O[b], and shift this half's x.
                        const float m_new = cmax == -INFINITY ? m_ref : fmaxf(m_ref, m_use + cmax);
                        const float scale = m_new == -INFINITY ? 1.f : fast_exp2(m_ref - m_new);
                        const float shift = (m_new == -INFINITY ? 0.f : m_new) - m_use;
                        m_ref = m_new;
                        l2.x *= scale;
                        l2.y *= scale;
                        l2b.x *= scale;
                        l2b.y *= scale;
                        const float2 ns2 = make_float2(-shift, -shift);
#pragma unroll
                        for (int e = 0; e < 32; ++e) x[e] = __fadd2_rn(x[e], ns2);
                        tmem_wait_st();
                        if (h > 0) {
#pragma unroll 1
                            for (int cc = 0; cc < 2; ++cc) {
                                uint32_t pk[16];
                                tmem_ld16(s_addr + 16u * cc, pk);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e)
                                    pk[e] = pack_bf16x2(bf16_lo(pk[e]) * scale, bf16_hi(pk[e]) * scale);
                                tmem_st16(s_addr + 16u * cc, pk);
                            }
                        }
                        if (mine > 0) {
#pragma unroll 1
                            for (int cc = 0; cc < 8; ++cc) {
                                uint32_t ro[16];
                                tmem_ld16(o_addr + 16u * cc, ro);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e) ro[e] = __float_as_uint(__uint_as_float(ro[e]) * scale);
                                tmem_st16(o_addr + 16u * cc, ro);
                            }
                        }
                        tmem_wait_st();
                    }
                    // P = exp2(x) as packed bf16: half h of the tile goes to columns [32 h, 32 h + 32) of
                    // the buffer, which this thread has already read
                    uint32_t pk[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const float2 pe = make_float2(fast_exp2(x[e].x), fast_exp2(x[e].y));
                        if (e & 1) l2b = __fadd2_rn(l2b, pe); else l2 = __fadd2_rn(l2, pe);
                        pk[e] = pack_bf16x2(pe.x, pe.y);
                    }
                    tmem_st16(s_addr + 32u * (uint32_t)h, *reinterpret_cast<uint32_t(*)[16]>(&pk[0]));
                    tmem_st16(s_addr + 32u * (uint32_t)h + 16u, *reinterpret_cast<uint32_t(*)[16]>(&pk[16]));
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();      // 128 arrivals on one barrier word would take turns; the warp's lanes are ordered here instead
                if (lane == 0) mbar_arrive(bar(kPFull0 + 2 * b));
                tr_work += trace_clock() - ts;
                if (lane == 0) trace_event(1 + warp, ev, 32);
            }
            if (!ok) break;
            const float l_sum = (l2.x + l2.y) + (l2b.x + l2b.y);
            load_q(it_next, q_next);        // in flight during the epilogue
            if (lane == 0) trace_event(1 + warp, ev, 33);
            // ---- epilogue.  The groups' (max, sum) go through columns 0-1 of their S buffers, which are
            // idle from the group's last P V until the next item's first Q K^T.
            if (mine > 0) {
                ok = mbar_wait_warp(bar(kPvDone0 + 2 * b), (uint32_t)pv_cnt & 1u, abort_flag, p.status, 34);
                if (!ok) break;
                ++pv_cnt;
                tc_fence_after();
                if (lane == 0) trace_event(1 + warp, ev, 34);
                // the V tile of the group's last tile goes back to the producers
                if (m == 0 && (!dual || b == 1))
                    mbar_arrive(bar(kRingEmpty0 + ring_pos_v(gt + (dual ? ntiles - 1 : b + 2 * (mine - 1))) % kRing));
            }
            tmem_st2(s_addr, __float_as_uint(m_ref), __float_as_uint(l_sum));
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kStats));
            ok = mbar_wait_warp(bar(kStats), (uint32_t)item_no & 1u, abort_flag, p.status, 35);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) trace_event(1 + warp, ev, 35);
            const size_t hq = (size_t)it.kv_head * G + g;
            const size_t prow = it.partial_row0 < 0 ? 0 : (size_t)it.partial_row0 + t;
            float w0, w1, lse2;          // weights of O[0] and O[1] in this thread's output row
            int c_begin, c_end;          // 32-column chunks of the row this thread writes
            if (dual) {
                const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
                w0 = b == 0 ? inv : 0.f;
                w1 = b == 1 ? inv : 0.f;
                lse2 = l_sum > 0.f ? m_ref + log2f(l_sum) : -INFINITY;
                c_begin = 0; c_end = 4;
            } else {
                // the two groups hold two KV splits of the same rows: merge them; group b writes value half b
                uint32_t x0, y0, x1, y1;
                tmem_ld2(lane_addr + kColS, x0, y0);
                tmem_ld2(lane_addr + kColS + 128u, x1, y1);
                tmem_wait_ld();
                const float m0 = __uint_as_float(x0), l0 = __uint_as_float(y0);
                const float m1 = __uint_as_float(x1), l1 = __uint_as_float(y1);
                const float M = fmaxf(m0, m1);
                const float a0 = l0 > 0.f ? fast_exp2(m0 - M) : 0.f;
                const float a1 = l1 > 0.f ? fast_exp2(m1 - M) : 0.f;
                const float L = a0 * l0 + a1 * l1;
                const float inv = L > 0.f ? 1.f / L : 0.f;
                w0 = a0 * inv;
                w1 = a1 * inv;
                lse2 = L > 0.f ? M + log2f(L) : -INFINITY;
                c_begin = 2 * b; c_end = 2 * b + 2;
            }
            const bool use0 = __any_sync(0xffffffffu, w0 != 0.f), use1 = __any_sync(0xffffffffu, w1 != 0.f);
            // A thread holds one row, but a row-per-thread store touches 32 lines per instruction: the
            // warp passes each 128-byte slice of its 32 rows through shared memory (its own rows of the Q
            // tile, which no MMA reads any more; 16-byte pieces XOR-swizzled by row) and writes whole lines.
            const int w4 = warp & 3;
            uint8_t* stage = smem + kOffQ + (dual ? b * kTileBytes : b * kHalfBytes) + w4 * 32 * 128;
            const int row_base = (dual ? 128 * b : 0) + 32 * w4;      // item row of the warp's first thread
            const bool final_out = it.partial_row0 < 0;
            auto flush = [&](int byte0) {      // byte0: offset of the slice inside an output row
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int row = 4 * i + (lane >> 3), pc = lane & 7;
                    const uint4 v = *reinterpret_cast<const uint4*>(stage + row * 128 + ((pc ^ (row & 7)) << 4));
                    const int ri = row_base + row, tt = ri / G, gg = ri % G;
                    if (tt < it.ntok) {
                        uint8_t* dst = final_out
                            ? reinterpret_cast<uint8_t*>(out + ((size_t)(it.q_row0 + tt) * Hq + (size_t)it.kv_head * G + gg) * kD)
                            : reinterpret_cast<uint8_t*>(p.partial_o + (((size_t)it.partial_row0 + tt) * G + gg) * kD);
                        *reinterpret_cast<uint4*>(dst + byte0 + pc * 16) = v;
                    }
                }
                __syncwarp();
            };
#pragma unroll 1
            for (int c = c_begin; c < c_end; ++c) {
                float acc[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] = 0.f;
                if (use0) {
                    uint32_t ro[32];
                    tmem_ld32(lane_addr + kColO + 32u * c, ro);
                    tmem_wait_ld();
                    if (w0 != 0.f) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) acc[e] = __uint_as_float(ro[e]) * w0;
                    }
                }
                if (use1) {
                    uint32_t ro[32];
                    tmem_ld32(lane_addr + kColO + 128u + 32u * c, ro);
                    tmem_wait_ld();
                    if (w1 != 0.f) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) acc[e] = fmaf(__uint_as_float(ro[e]), w1, acc[e]);
                    }
                }
                uint8_t* mine_row = stage + lane * 128;
                if (final_out) {
                    // 32 columns -> 64 bytes of bf16: pieces 4 (c & 1) .. + 3 of a 64-column slice
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<uint4*>(mine_row + ((((c & 1) * 4 + k) ^ (lane & 7)) << 4)) =
                            make_uint4(pack_bf16x2(acc[8 * k], acc[8 * k + 1]), pack_bf16x2(acc[8 * k + 2], acc[8 * k + 3]),
                                       pack_bf16x2(acc[8 * k + 4], acc[8 * k + 5]), pack_bf16x2(acc[8 * k + 6], acc[8 * k + 7]));
                    if (c & 1) flush((c >> 1) * 128);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        *reinterpret_cast<uint4*>(mine_row + ((k ^ (lane & 7)) << 4)) =
                            make_uint4(__float_as_uint(acc[4 * k]), __float_as_uint(acc[4 * k + 1]),
                                       __float_as_uint(acc[4 * k + 2]), __float_as_uint(acc[4 * k + 3]));
                    flush(c * 128);
                }
            }
            if (row_valid && (dual || b == 0)) {
                if (it.partial_row0 < 0) {
                    if (lse != nullptr) lse[(size_t)(it.q_row0 + t) * Hq + hq] = lse2 * kLn2;
                } else {
                    p.partial_lse[prow * G + g] = lse2;
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kOFree));
            if (lane == 0) trace_event(1 + warp, ev, 36);
            cnt += mine;
            gt += ntiles;
        }
        if ((threadIdx.x & 127) == 0) {
            trace_set(b ? 15 : 11, tr_wait);
            if (b == 0) { trace_set(12, tr_work); trace_set(13, tr_tiles); }
        }
    }

    // common exit: every role gets here, then the allocating warp releases tensor memory
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace tc

}  // namespace asynclm
