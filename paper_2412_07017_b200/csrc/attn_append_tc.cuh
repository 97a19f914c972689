// Tensor-core attention for interrupt spans (tcgen05 MMA with accumulators in tensor memory).
//
// An interrupt span is a block of new tokens appended to one sequence (paper Section 3.2); in the
// next decoding step (Section 5.3) every token of the span attends to the whole cached context and
// causally to the span itself.  With G query heads per kv head, a span of q tokens gives G*q query
// rows against the same K/V, which is a dense contraction: rows are packed 128 to a tile
// (row m = token m / G, head m % G) and S = Q K^T and O += P V run on the tensor cores.
//
// One persistent CTA per SM, ten warps:
//   warps 0-3, 4-7  two softmax groups, one thread per query row each.  Group b takes the KV tiles
//                   j = b, b+2, ... of an item and owns S[b], P[b] and O[b]: softmax on S read from
//                   tensor memory, P written to shared memory as bf16, lazy rescaling of O[b].  The
//                   two running (max, sum, O) states are merged in the epilogue like two KV splits.
//   warps 8, 10     producers of the K ring and of the V ring: 16-byte cp.async copies (fully coalesced,
//                   two 256-byte rows per warp instruction) that write the 128-byte-swizzled operand
//                   layout directly and complete on the stage's mbarrier; rows behind the last key are
//                   zero-filled.  (Tiled TMA would need 32 boxes of 2 KiB per 128-key tile, and the
//                   measured cost of about 90 cycles per small bulk/TMA copy made that the bottleneck.)
//                   The two rings run independently so that a K tile never queues behind a V stage
//                   that is still waiting for its P V to finish.
//   warps 9, 11     one thread each issues the Q K^T MMAs and the P V MMAs.  tcgen05.mma issue blocks
//                   once a few MMAs are queued, so a single issuing thread alternates between being
//                   blocked and doing its barrier bookkeeping while the tensor pipe idles; with two
//                   issuers one's bookkeeping hides behind the other's MMAs.  Warp 9 owns the
//                   tensor-memory allocation.
// While one group runs the softmax of tile j the tensor core computes Q K^T of tile j+1 and P V of
// tile j-1 for the other group.  All hand-offs are mbarriers with bounded waits; a wait that runs
// out sets the plan's status word and a CTA-wide abort flag, every role falls through to the common
// exit, and the tensor memory is released there.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace tc {

constexpr int kThreads = 384;
constexpr int kProducerWarpK = 8, kMmaWarp = 9, kProducerWarpV = 10, kMmaWarpPV = 11;
constexpr int kD = 128;
constexpr int kTile = 128;                       // keys per KV tile and query rows per tile
constexpr int kKS = 2, kVS = 2;                  // ring depths
constexpr uint32_t kHalfBytes = 128 * 128;       // one 64-value half of a 128-row tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;  // 32 KiB
constexpr float kRescaleThreshold = 8.f;
constexpr long long kWaitCycles = 2000000000ll;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffP = kOffQ + kTileBytes;          // P[0], P[1]
constexpr uint32_t kOffK = kOffP + 2 * kTileBytes;
constexpr uint32_t kOffV = kOffK + kKS * kTileBytes;
constexpr uint32_t kOffBar = kOffV + kVS * kTileBytes;
enum Bar { kQFull = 0, kStats, kOFree, kPFull0, kPFull1, kPvDone0, kPvDone1, kSFull0, kSFull1, kKFull0,
           kKEmpty0 = kKFull0 + kKS, kVFull0 = kKEmpty0 + kKS, kVEmpty0 = kVFull0 + kVS,
           kMmaDrain = kVEmpty0 + kVS, kMmaDrain2, kNumBars };
constexpr uint32_t kOffTmemPtr = kOffBar + 8 * kNumBars;
constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
constexpr uint32_t kSmemBytes = kOffAbort + 8 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");

// tensor memory columns
constexpr uint32_t kColS = 0;      // S[0], S[1]: 128 columns each
constexpr uint32_t kColO = 256;    // O[0], O[1]: 128 columns each
constexpr uint32_t kTmemCols = 512;

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
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

struct TItem {
    int kv0, kv_end;      // key range of the item after causal clipping (kv_end == 0: no item)
    int q_row0, ntok, kv_limit0, kv_head, partial_base, chunk, page0;
};

__device__ __forceinline__ TItem load_titem(const DevPlan& p, int ii, int i1) {
    TItem r{0, 0, 0, 0, 0, 0, -1, 0, 0};
    if (ii < i1) {
        const Item it = p.items[ii];
        const Unit u = p.units[it.unit];
        r.kv0 = it.kv0;
        r.kv_end = min(it.kv1, u.kv_limit0 + u.ntok - 1);
        r.q_row0 = u.q_row0;
        r.ntok = u.ntok;
        r.kv_limit0 = u.kv_limit0;
        r.kv_head = u.kv_head;
        r.partial_base = u.partial_base;
        r.chunk = it.chunk;
        r.page0 = u.page_base + it.kv0 / kPage;
    }
    return r;
}

// Register shares of the fused kernel's tensor-core phase (512 threads launched with 128 each):
// softmax warps 0-7, the producer/MMA warpgroup 8-11, and warps 12-15, which idle in this phase.
constexpr int kRegsSoftmaxFused = 168, kRegsIssueFused = 80, kRegsIdleFused = 24;
static_assert(256 * kRegsSoftmaxFused + 128 * kRegsIssueFused + 128 * kRegsIdleFused <= 65536, "register split");

// The whole kernel body.  FUSED: called by all 16 warps of the fused kernel (warps 11-15 only take
// part in the CTA-wide barriers), with `smem` 1024-byte aligned.
template <int G, bool FUSED>
__device__ __forceinline__ void tc_body(const DevPlan& p, const __nv_bfloat16* __restrict__ q,
                                        const __nv_bfloat16* __restrict__ pool,
                                        __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                        uint8_t* smem) {
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_ptr = (volatile uint32_t*)(smem + kOffTmemPtr);
    volatile int* abort_flag = (volatile int*)(smem + kOffAbort);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int Hq = p.num_q_heads, Hkv = p.num_kv_heads;
    const int i0 = p.cta_indptr_tensor[blockIdx.x], i1 = p.cta_indptr_tensor[blockIdx.x + 1];

    if (threadIdx.x == 0) {
        mbar_init(bar(kQFull), 256);
        mbar_init(bar(kStats), 256);
        mbar_init(bar(kOFree), 256);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(kPFull0 + b), 128);
            mbar_init(bar(kPvDone0 + b), 1);
            mbar_init(bar(kSFull0 + b), 1);
        }
        for (int s = 0; s < kKS; ++s) { mbar_init(bar(kKFull0 + s), 32); mbar_init(bar(kKEmpty0 + s), 1); }
        for (int s = 0; s < kVS; ++s) { mbar_init(bar(kVFull0 + s), 32); mbar_init(bar(kVEmpty0 + s), 1); }
        mbar_init(bar(kMmaDrain), 1);
        mbar_init(bar(kMmaDrain + 1), 1);
        *abort_flag = 0;
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
    // Launched with programmatic serialization: everything above overlapped the tail of the append
    // kernel; from here on the pool is read.  Once every CTA has passed this point the CUDA-core
    // kernel behind this one may start on SMs that become free.
    pdl_wait();
    if constexpr (!FUSED) pdl_trigger();

    if (warp >= 12) {
        if constexpr (FUSED) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIdleFused));
    } else if (warp >= 8) {
      if constexpr (FUSED) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssueFused));
      if (warp == kProducerWarpK || warp == kProducerWarpV) {
        // ------------------------------------------------------------------ producer warps
        const int which = warp == kProducerWarpV ? 1 : 0;       // 0: K ring, 1: V ring
        const int stages = which ? kVS : kKS;
        const int full0 = which ? kVFull0 : kKFull0, empty0 = which ? kVEmpty0 : kKEmpty0;
        const uint32_t ring = sbase + (which ? kOffV : kOffK);
        auto load_pages = [&](const TItem& it, int first_page) {
            const int npg = (it.kv_end - it.kv0 + kPage - 1) / kPage;
            const int idx = first_page + lane;
            return idx < npg ? __ldg(p.page_indices + it.page0 + idx) : 0;
        };
        constexpr int kPagesPerTile = kTile / kPage;          // 8
        constexpr int kGroupTiles = 32 / kPagesPerTile;       // 4
        bool ok = true;
        int n = 0;                                             // tiles issued so far
        TItem cur = load_titem(p, i0, i1), nxt = load_titem(p, i0 + 1, i1);
        int pages_cur = cur.kv_end > 0 ? load_pages(cur, 0) : 0;
        for (int ii = i0; cur.kv_end > 0 && ok; ++ii) {
            const TItem after = load_titem(p, ii + 2, i1);
            const int ntiles = (cur.kv_end - cur.kv0 + kTile - 1) / kTile;
            for (int t0 = 0; t0 < ntiles && ok; t0 += kGroupTiles) {
                int pages_nxt = 0;
                if (t0 + kGroupTiles < ntiles) pages_nxt = load_pages(cur, (t0 + kGroupTiles) * kPagesPerTile);
                else if (nxt.kv_end > 0) pages_nxt = load_pages(nxt, 0);
                const int t1 = min(t0 + kGroupTiles, ntiles);
                for (int t = t0; t < t1 && ok; ++t, ++n) {
                    const int rows = min(kTile, cur.kv_end - (cur.kv0 + t * kTile));
                    const int npages = (rows + kPage - 1) / kPage;
                    const int s = n % stages;
                    ok = mbar_wait_warp(bar(empty0 + s), ((uint32_t)(n / stages) & 1u) ^ 1u, abort_flag, p.status, 11 + which);
                    if (!ok) break;
                    // lane -> 16-byte chunk c of row 2*rr + (lane >> 4) of each page: a warp instruction
                    // moves two whole 256-byte rows
                    const int c = lane & 15;
                    const uint32_t dst_half = ring + s * kTileBytes + (uint32_t)(c >> 3) * kHalfBytes;
                    for (int pg = 0; pg < npages; ++pg) {
                        const int64_t page = __shfl_sync(0xffffffffu, pages_cur, (t - t0) * kPagesPerTile + pg);
                        const uint8_t* src_page = reinterpret_cast<const uint8_t*>(
                            pool + pool_row_offset(page, which, cur.kv_head, 0, Hkv, kD));
#pragma unroll
                        for (int rr = 0; rr < kPage / 2; ++rr) {
                            const int slot = rr * 2 + (lane >> 4);
                            const int row = pg * kPage + slot;
                            cp_async16(dst_half + (uint32_t)row * 128u + (uint32_t)(((c & 7) ^ (row & 7)) << 4),
                                       src_page + slot * (kD * 2) + c * 16, row < rows ? 16u : 0u);
                        }
                    }
                    cp_async_arrive(bar(full0 + s));
                }
                pages_cur = pages_nxt;
            }
            cur = nxt;
            nxt = after;
        }
        if (!ok) {
            // aborted: let the loads already issued land before shared memory goes away
            const long long t0 = clock64();
            for (int k = max(0, n - stages); k < n; ++k)
                while (!mbar_try_wait(bar(full0 + k % stages), (uint32_t)(k / stages) & 1u) && clock64() - t0 < kWaitCycles) {}
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ Q K^T issuer
        if (lane == 0) {
            bool ok = true;
            int gt = 0;               // KV tiles issued so far (all items): ring position
            int cnt[2] = {0, 0};      // tiles handed to each softmax group so far: S/P phase
            int item_no = 0;
            TItem it_next = load_titem(p, i0, i1);
            for (int ii = i0; ii < i1 && ok; ++ii, ++item_no) {
                const TItem it = it_next;
                it_next = load_titem(p, ii + 1, i1);      // in flight while this item runs
                const int ntiles = (it.kv_end - it.kv0 + kTile - 1) / kTile;
                ok = mbar_wait(bar(kQFull), (uint32_t)item_no & 1u, abort_flag, p.status, 22);
                if (ok) tc_fence_after();
                // S[b] <- Q K_j^T for tile j of the item (b = j & 1); S[b] is free once group b has turned
                // its previous tile into P
                for (int j = 0; j < ntiles && ok; ++j) {
                    const int g = gt + j, b = j & 1;
                    const int s = g % kKS;
                    if (j >= 2)
                        ok = mbar_wait(bar(kPFull0 + b), (uint32_t)(cnt[b] + (j >> 1) - 1) & 1u, abort_flag, p.status, 23);
                    ok = ok && mbar_wait(bar(kKFull0 + s), (uint32_t)(g / kKS) & 1u, abort_flag, p.status, 21);
                    if (!ok) break;
                    tc_fence_after();
                    const int npg = (min(kTile, it.kv_end - (it.kv0 + j * kTile)) + kPage - 1) / kPage;
                    const uint32_t idesc = instr_desc(16u * (uint32_t)npg, 0);
                    const uint32_t d = tmem + kColS + 128u * (uint32_t)b;
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint32_t off = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                        mma_f16(d, smem_desc(sbase + kOffQ + off, 16, 1024),
                                smem_desc(sbase + kOffK + s * kTileBytes + off, 16, 1024), idesc, ks > 0);
                    }
                    mma_commit(bar(kKEmpty0 + s));
                    mma_commit(bar(kSFull0 + b));
                }
                gt += ntiles;
                cnt[0] += (ntiles + 1) >> 1;
                cnt[1] += ntiles >> 1;
            }
            // make sure nothing is still running on the tensor core before tensor memory is released
            mma_commit(bar(kMmaDrain));
            const long long t0 = clock64();
            while (!mbar_try_wait(bar(kMmaDrain), 0) && clock64() - t0 < kWaitCycles) {}
        }
        __syncwarp();
      } else if (warp == kMmaWarpPV) {
        // ------------------------------------------------------------------ P V issuer
        if (lane == 0) {
            bool ok = true;
            int gt = 0;
            int cnt[2] = {0, 0};
            int item_no = 0;
            const uint32_t idesc_pv = instr_desc(128, 1);
            TItem it_next = load_titem(p, i0, i1);
            for (int ii = i0; ii < i1 && ok; ++ii, ++item_no) {
                const TItem it = it_next;
                it_next = load_titem(p, ii + 1, i1);
                const int ntiles = (it.kv_end - it.kv0 + kTile - 1) / kTile;
                // O[b] (+)= P_j V_j: P[b] comes from group b, V from the ring; the first P V into each
                // accumulator of an item overwrites it, so the previous item's epilogue must be done
                for (int j = 0; j < ntiles && ok; ++j) {
                    const int g = gt + j, b = j & 1;
                    const int s = g % kVS;
                    ok = mbar_wait(bar(kPFull0 + b), (uint32_t)(cnt[b] + (j >> 1)) & 1u, abort_flag, p.status, 26) &&
                         mbar_wait(bar(kVFull0 + s), (uint32_t)(g / kVS) & 1u, abort_flag, p.status, 24);
                    if (ok && j == 0 && item_no > 0)
                        ok = mbar_wait(bar(kOFree), (uint32_t)(item_no - 1) & 1u, abort_flag, p.status, 25);
                    if (!ok) break;
                    tc_fence_after();
                    const int npg = (min(kTile, it.kv_end - (it.kv0 + j * kTile)) + kPage - 1) / kPage;
                    for (int ks = 0; ks < npg; ++ks) {
                        const uint32_t poff = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                        mma_f16(tmem + kColO + 128u * (uint32_t)b,
                                smem_desc(sbase + kOffP + b * kTileBytes + poff, 16, 1024),
                                smem_desc(sbase + kOffV + s * kTileBytes + (uint32_t)ks * 2 * 1024u, kHalfBytes, 1024),
                                idesc_pv, (j > 1 || ks > 0) ? 1u : 0u);
                    }
                    mma_commit(bar(kVEmpty0 + s));
                    mma_commit(bar(kPvDone0 + b));
                }
                gt += ntiles;
                cnt[0] += (ntiles + 1) >> 1;
                cnt[1] += ntiles >> 1;
            }
            mma_commit(bar(kMmaDrain + 1));
            const long long t0 = clock64();
            while (!mbar_try_wait(bar(kMmaDrain + 1), 0) && clock64() - t0 < kWaitCycles) {}
        }
        __syncwarp();
      }
    } else {
        if constexpr (FUSED) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmaxFused));
        // ------------------------------------------------------------------ softmax / epilogue groups
        const int b = warp >> 2;                   // softmax group
        const int m = threadIdx.x & 127;           // query row of the tile = tensor-memory lane
        const int t = m / G, g = m % G;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t s_addr = lane_addr + kColS + 128u * (uint32_t)b;
        const uint32_t o_addr = lane_addr + kColO + 128u * (uint32_t)b;
        uint8_t* p_smem = smem + kOffP + b * kTileBytes;
        // (max, sum) of each group and row for the epilogue live at the start of that group's P buffer:
        // P[b] is idle from the group's last P.V until the next item's first Q K^T, which cannot be
        // issued before every thread has read the statistics and staged the next Q.
        float2* stats0 = reinterpret_cast<float2*>(smem + kOffP);
        float2* stats1 = reinterpret_cast<float2*>(smem + kOffP + kTileBytes);
        const float qscale = p.sm_scale * kLog2e;
        int gt = 0;          // KV tiles before this item (all groups)
        int cnt = 0;         // tiles this group has processed before this item
        int item_no = 0;
        bool ok = true;
        // This thread's share of an item's Q: row m, the 8 chunks (16 bytes each) of value half b.  The
        // next item's descriptor and Q rows are fetched while the current item runs.
        auto load_q = [&](const TItem& x, uint4 (&w)[8]) {
            const bool valid = x.kv_end > 0 && t < x.ntok;
            const uint4* src = reinterpret_cast<const uint4*>(
                q + ((size_t)(x.q_row0 + t) * Hq + (size_t)x.kv_head * G + g) * kD) + 8 * b;
#pragma unroll
            for (int c = 0; c < 8; ++c) w[c] = valid ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
        };
        TItem it_next = load_titem(p, i0, i1);
        uint4 q_next[8];
        load_q(it_next, q_next);
        for (int ii = i0; ii < i1 && ok; ++ii, ++item_no) {
            const TItem it = it_next;
            const int ntiles = (it.kv_end - it.kv0 + kTile - 1) / kTile;
            const bool row_valid = t < it.ntok;
            // ---- stage Q with the 128-byte swizzle the MMA descriptor expects
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(smem + kOffQ + b * kHalfBytes + m * 128 + ((c ^ (m & 7)) << 4)) = q_next[c];
            fence_async_smem();
            mbar_arrive(bar(kQFull));
            it_next = load_titem(p, ii + 1, i1);
            load_q(it_next, q_next);
            const int lim_row = row_valid ? min(it.kv_limit0 + t, it.kv_end) : 0;   // keys [0, lim_row) visible
            float m_ref = -INFINITY, l_sum = 0.f;
            int mine = 0;                                                          // tiles of this group so far
            for (int j = b; j < ntiles && ok; j += 2, ++mine) {
                const int base = it.kv0 + j * kTile;
                const int vis = max(0, min(kTile, lim_row - base));     // visible columns of this row
                ok = mbar_wait_warp(bar(kSFull0 + b), (uint32_t)(cnt + mine) & 1u, abort_flag, p.status, 31);
                if (!ok) break;
                tc_fence_after();
                const bool full_tile = __all_sync(0xffffffffu, vis == kTile);
                if (mine == 0) {
                    // first tile of the group: the reference maximum is this tile's row maximum
                    float tmax = -INFINITY;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tmem_ld32(s_addr + 32u * c, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            tmax = fmaxf(tmax, (full_tile || c * 32 + e < vis) ? __uint_as_float(r[e]) : -INFINITY);
                    }
                    m_ref = tmax * qscale;     // qscale > 0: the maximum commutes with the scaling
                } else {
                    // P[b] and O[b] are still in use by the P.V of this group's previous tile
                    ok = mbar_wait_warp(bar(kPvDone0 + b), (uint32_t)(cnt + mine - 1) & 1u, abort_flag, p.status, 32);
                    if (!ok) break;
                    tc_fence_after();
                }
                // P = exp2(S * scale - m_ref) as bf16 into shared memory (A operand of P.V).  The
                // reference maximum is only moved when some score exceeds it by the threshold; then O[b]
                // and the running sum are rescaled and the tile is redone.
                float l_tile = 0.f;
#pragma unroll 1
                for (int attempt = 0; attempt < 2; ++attempt) {
                    const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
                    float tmax = -INFINITY;
                    l_tile = 0.f;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tmem_ld32(s_addr + 32u * c, r);
                        tmem_wait_ld();
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            float s0 = __uint_as_float(r[e]), s1 = __uint_as_float(r[e + 1]);
                            if (!full_tile) {
                                if (c * 32 + e >= vis) s0 = -INFINITY;
                                if (c * 32 + e + 1 >= vis) s1 = -INFINITY;
                            }
                            tmax = fmaxf(tmax, fmaxf(s0, s1));
                            const float p0 = fast_exp2(fmaf(s0, qscale, -m_use));
                            const float p1 = fast_exp2(fmaf(s1, qscale, -m_use));
                            l_tile += p0 + p1;
                            pk[e >> 1] = pack_bf16x2(p0, p1);
                        }
                        // columns [32c, 32c+32) = 4 chunks of 8 keys: key half c >> 1, chunks (c & 1) * 4 ..
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int cc = (c & 1) * 4 + k;
                            *reinterpret_cast<uint4*>(p_smem + (c >> 1) * kHalfBytes + m * 128 + ((cc ^ (m & 7)) << 4)) =
                                make_uint4(pk[4 * k], pk[4 * k + 1], pk[4 * k + 2], pk[4 * k + 3]);
                        }
                    }
                    tmax *= qscale;
                    if (attempt == 1 || !__any_sync(0xffffffffu, tmax > m_ref + kRescaleThreshold)) break;
                    const float m_new = fmaxf(m_ref, tmax);
                    const float scale = m_new == -INFINITY ? 1.f : fast_exp2(m_ref - m_new);
                    m_ref = m_new;
                    l_sum *= scale;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tmem_ld32(o_addr + 32u * c, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * scale);
                        tmem_st32(o_addr + 32u * c, r);
                    }
                    tmem_wait_st();
                }
                l_sum += l_tile;
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar(kPFull0 + b));
            }
            if (!ok) break;
            // ---- epilogue: merge the two groups' states, group b writes value half b of every row
            if (mine > 0) {
                ok = mbar_wait_warp(bar(kPvDone0 + b), (uint32_t)(cnt + mine - 1) & 1u, abort_flag, p.status, 34);
                if (!ok) break;
                tc_fence_after();
            }
            (b == 0 ? stats0 : stats1)[m] = make_float2(m_ref, l_sum);
            mbar_arrive(bar(kStats));
            ok = mbar_wait_warp(bar(kStats), (uint32_t)item_no & 1u, abort_flag, p.status, 35);
            if (!ok) break;
            const float2 st0 = stats0[m], st1 = stats1[m];
            const float M = fmaxf(st0.x, st1.x);
            const float a0 = st0.y > 0.f ? fast_exp2(st0.x - M) : 0.f;
            const float a1 = st1.y > 0.f ? fast_exp2(st1.x - M) : 0.f;
            const float L = a0 * st0.y + a1 * st1.y;
            const float inv = L > 0.f ? 1.f / L : 0.f;
            const float w0 = a0 * inv, w1 = a1 * inv;
            const float lse2 = L > 0.f ? M + log2f(L) : -INFINITY;
            const size_t hq = (size_t)it.kv_head * G + g;
            const size_t prow = it.partial_base < 0 ? 0 : (size_t)it.partial_base + (size_t)it.chunk * it.ntok + t;
            const bool use0 = __any_sync(0xffffffffu, w0 != 0.f), use1 = __any_sync(0xffffffffu, w1 != 0.f);
#pragma unroll 1
            for (int c = 2 * b; c < 2 * b + 2; ++c) {
                float acc[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] = 0.f;
                if (use0) {
                    uint32_t r[32];
                    tmem_ld32(lane_addr + kColO + 32u * c, r);
                    tmem_wait_ld();
                    if (w0 != 0.f) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) acc[e] = __uint_as_float(r[e]) * w0;
                    }
                }
                if (use1) {
                    uint32_t r[32];
                    tmem_ld32(lane_addr + kColO + 128u + 32u * c, r);
                    tmem_wait_ld();
                    if (w1 != 0.f) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) acc[e] = fmaf(__uint_as_float(r[e]), w1, acc[e]);
                    }
                }
                if (row_valid) {
                    if (it.partial_base < 0) {
                        uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)(it.q_row0 + t) * Hq + hq) * kD + c * 32);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            dst[k] = make_uint4(pack_bf16x2(acc[8 * k], acc[8 * k + 1]), pack_bf16x2(acc[8 * k + 2], acc[8 * k + 3]),
                                                pack_bf16x2(acc[8 * k + 4], acc[8 * k + 5]), pack_bf16x2(acc[8 * k + 6], acc[8 * k + 7]));
                    } else {
                        float4* dst = reinterpret_cast<float4*>(p.partial_o + (prow * G + g) * kD + c * 32);
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            dst[k] = make_float4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
                    }
                }
            }
            if (row_valid && b == 0) {
                if (it.partial_base < 0) {
                    if (lse != nullptr) lse[(size_t)(it.q_row0 + t) * Hq + hq] = lse2 * kLn2;
                } else {
                    p.partial_lse[prow * G + g] = lse2;
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kOFree));
            gt += ntiles;
            cnt += mine;
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
