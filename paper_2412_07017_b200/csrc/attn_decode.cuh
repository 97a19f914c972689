// Warp-level attention for decode rows (and spans too short for the tcgen05 path).
//
// Each new token attends to its sequence's whole cached context plus its own span up to itself
// (paper Section 3.2 / 5.3: interrupt tokens are appended to the context and processed in the next
// decoding step, next to the other sequences' one-token decodes).  This path has to be bound by HBM
// bandwidth: every K/V row is read once and used by the G query heads that share the kv head, i.e.
// G multiply-adds per byte, far below the machine's ridge.  Doing those multiply-adds on the fp32
// pipes costs an unpack and two FMAs per bf16 pair and made the path instruction-bound, so the two
// small contractions of a page run on warp-level tensor instructions (mma.sync m16n8k16) with the
// KEYS on the M axis, which wastes nothing on padding query rows:
//     S^T [16 keys x 8 columns]   = K_page [16 x d]      . Q^T [d x 8]        (d / 16 instructions)
//     O^T [d x 8 columns]        += V_page^T [d x 16]    . P^T [16 x 8]       (d / 16 instructions)
// A column is one (token, head) pair of the unit: up to 8 / G consecutive tokens times the G heads
// of the kv head; unused columns carry zeros.  About 70 warp instructions per page instead of 700.
//
// Structure: one persistent CTA per SM walks the item list the planner gave it.  A producer warp
// streams the items' pages into a shared-memory ring of 128-key stages, one tiled TMA copy per
// (page, kv head) that brings the K block and the V block together and lands them with the
// 128-byte swizzle that makes ldmatrix conflict-free; a small descriptor and the unit's query rows
// travel with each stage.  Eight consumer warps take one page of a stage each: ldmatrix, the two
// contractions, softmax against a lazily moved reference maximum on the accumulator fragment
// (4 values per thread), P transposed in registers (movmatrix) into the B operand.  At the end of
// an item each consumer warp drops its state into its own page slot of the item's last stage and
// goes straight on to the next item; an epilogue warp combines the eight states, writes final bf16
// output or the fp32 partial of a chunk, and hands the stage back to the producer.  When the chunk
// belongs to a unit whose keys were split, the epilogue warp also counts it in (one atomic add per
// chunk); the CTA that brings the count to the number of chunks merges the unit's partial results
// in chunk order on a merge warp of its own, so no merge kernel has to follow and no consumer ever
// waits for another warp.
//
// Every wait is bounded: a wait that runs out sets the plan's device status word and a CTA-wide
// abort flag, after which all loops fall through and the kernel returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace dec {

constexpr int kWarps = 8;                    // consumer warps: one page of a 128-key stage each
constexpr int kProducerWarp = kWarps;        // the warp behind them streams the pages
constexpr int kEpilogueWarp = kWarps + 1;    // combines the consumers' states at the end of an item
constexpr int kMergeWarp = kWarps + 2;       // merges the chunks of a split unit once all have arrived
constexpr int kFetchWarp = kWarps + 3;       // claims the next chunk and fetches its record and page ids
constexpr int kThreads = (kWarps + 4) * 32;  // consumers, producer, epilogue, merge, fetch
constexpr int kMergeReqs = 4;                // merge requests in flight between the last two
constexpr int kMaxStages = 6;
constexpr int kHandoffs = kMaxStages + 2;    // item hand-offs in flight: a stage each, so at most kMaxStages
constexpr int kCols = 8;                     // (token, head) columns of a unit: the N of the MMAs
constexpr int kTileTok = kWarps * kPage;     // keys per ring stage
constexpr float kRescaleThreshold = 8.f;     // log2 units a score may exceed the reference max by
constexpr long long kWaitCycles = 2000000000ll;

constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagEnd = 4;

struct TileDesc {
    int32_t flags;
    int32_t rows;         // keys of this stage that some column may see
    int32_t lim0;         // keys of this stage that column 0's token sees (may be <= 0 or > rows)
    int32_t ntok;         // tokens of the unit
    int32_t out_row;      // global token row of the unit's first token
    int32_t kv_head;
    int32_t partial_row;  // -1: final output
    int32_t unit;         // the unit the item is a chunk of, its number of chunks and the partial row of
    int32_t n_chunks;     // its chunk 0 (for the merge of a split unit)
    int32_t partial_base;
    int32_t stage;        // hand-off only: the stage that holds the consumers' states
    int32_t pad;
};

// What the fetch warp hands to the producer: the next item's record and its first 32 page ids.
struct NextItem {
    int32_t work[12];     // a Work record; work[1] (kv_end) == 0: nothing is left
    int32_t pages[32];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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
// Bounded wait.  Returns false (and raises the abort flag) if the phase did not complete in time
// or if another thread already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status, int code) {
    if (*abort_flag) return false;
    if (mbar_try_wait(bar, parity)) return true;
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// One tiled TMA copy fetches the K block and the V block of a (page, kv head).  The pool is
// described to the TMA unit as a 5-D tensor
//     (64 values, 16 slots, d / 64 halves of a row, Hkv heads, 2 * pages [page * 2 + K|V])
// and the box spans (64, 16, d / 64, 1, 2): two separate 16 x d blocks of global memory that land
// back to back in shared memory as [K|V][half][slot][64 values], every 128-byte row swizzled by its
// slot (16-byte piece c of slot s sits at piece c ^ (s & 7)).  No multicast.
__device__ __forceinline__ void tma_page_kv(uint32_t dst, const CUtensorMap* map, int kv_head, int page, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(0), "r"(0), "r"(0), "r"(kv_head), "r"(2 * page), "r"(bar) : "memory");
}

// Four 8x8 b16 matrices; lane l gives the address of row l % 8 of matrix l / 8; thread (g, t) =
// (lane / 4, lane % 4) receives elements [g][2t], [g][2t+1] of each (transposed: [2t][g], [2t+1][g]).
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// Transpose of an 8x8 b16 matrix held one row per four threads.
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// D (16x8, fp32) += A (16x16, bf16, row) . B (16x8, bf16, col).  Thread (g, t) holds
//   A: [g][2t..], [g+8][2t..], [g][2t+8..], [g+8][2t+8..]   B: [2t..][g], [2t+8..][g]
//   D: [g][2t], [g][2t+1], [g+8][2t], [g+8][2t+1]
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int D>
struct Geometry {
    static constexpr int HALVES = D / 64;                       // 128-byte pieces of a K or V row
    static constexpr int BLOCK_BYTES = kPage * D * 2;           // one (page, K|V, head) block
    static constexpr int PAGE_BYTES = 2 * BLOCK_BYTES;          // K block + V block: one TMA copy
    static constexpr int STAGE_BYTES = kWarps * PAGE_BYTES;     // 64 KiB at d = 128
    static constexpr int Q_BYTES = kCols * D * 2;               // the unit's query rows, [column][d]
    static constexpr int KSTEPS = D / 16;
    // merge area of a warp inside its page slot: O^T as [column][d + 4] fp32 (the pad keeps the
    // fragment stores conflict-free), then the columns' reference maxima and sums
    static constexpr int O_STRIDE = D + 4;
    static constexpr int STATE_FLOATS = kCols * O_STRIDE + 2 * kCols;
    static_assert(STATE_FLOATS * 4 <= PAGE_BYTES, "a warp's merge state must fit its page slot");
};

template <int D>
size_t smem_bytes(int stages) {
    using Geo = Geometry<D>;
    return (size_t)stages * (Geo::STAGE_BYTES + Geo::Q_BYTES + sizeof(TileDesc) + 16) +
           (size_t)(kHandoffs + kMergeReqs) * (sizeof(TileDesc) + 8) + kMergeReqs * 8 + sizeof(NextItem) + 16 +
           16 + 1024;
}

// The epilogue warp's loop (see the file comment): combine the consumers' states of a finished item,
// write the result, give the stage back, and pass a completed split unit on to the merge warp.
template <int D, int G>
__device__ __forceinline__ void epilogue_loop(const DevPlan& p, __nv_bfloat16* __restrict__ out,
                                              float* __restrict__ lse, uint8_t* stage_base,
                                              const TileDesc* handoff, TileDesc* merge_req, uint32_t empty0,
                                              uint32_t done0, uint32_t req0, uint32_t reqfree0,
                                              volatile int* abort_flag) {
    using Geo = Geometry<D>;
    const int lane = threadIdx.x & 31;
    const int Hq = p.num_q_heads;
    int n_req = 0;
    auto post = [&](const TileDesc& d) {      // to the merge warp; false if the wait for a free slot ran out
        const int j = n_req % kMergeReqs;
        if (!mbar_wait(reqfree0 + 8 * j, ((uint32_t)(n_req / kMergeReqs) & 1u) ^ 1u, abort_flag, p.status, 4)) return false;
        if (lane == 0) {
            merge_req[j] = d;
            mbar_arrive(req0 + 8 * j);
        }
        ++n_req;
        return true;
    };
    pdl_wait();      // outputs may be written only after the kernel in front has completed
    for (int k = 0;; ++k) {
        const int h = k % kHandoffs;
        if (!mbar_wait(done0 + 8 * h, (uint32_t)(k / kHandoffs) & 1u, abort_flag, p.status, 3)) break;
        const TileDesc d = handoff[h];
        if (d.flags & kFlagEnd) {
            post(d);
            break;
        }
        const uint8_t* stage = stage_base + (size_t)d.stage * Geo::STAGE_BYTES;
        const int ncols = d.ntok * G;
        // four consecutive values of one column per lane and pass; the eight warps' copies are read
        // with independent loads
        for (int e = 4 * lane; e < ncols * D; e += 128) {
            const int col = e / D, dd = e % D;
            float mw[kWarps], lw[kWarps];
            float4 ov[kWarps];
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float* sw = reinterpret_cast<const float*>(stage + (size_t)w * Geo::PAGE_BYTES);
                mw[w] = sw[kCols * Geo::O_STRIDE + col];
                lw[w] = sw[kCols * Geo::O_STRIDE + kCols + col];
                ov[w] = *reinterpret_cast<const float4*>(sw + (size_t)col * Geo::O_STRIDE + dd);
                M = fmaxf(M, mw[w]);
            }
            float L = 0.f;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float wgt = mw[w] == -INFINITY ? 0.f : fast_exp2(mw[w] - M);
                if (wgt != 0.f) {      // a warp without a visible key left nothing meaningful behind
                    L = fmaf(lw[w], wgt, L);
                    a.x = fmaf(ov[w].x, wgt, a.x); a.y = fmaf(ov[w].y, wgt, a.y);
                    a.z = fmaf(ov[w].z, wgt, a.z); a.w = fmaf(ov[w].w, wgt, a.w);
                }
            }
            const float inv = L > 0.f ? 1.f / L : 0.f;
            const float lse2 = L > 0.f ? M + log2f(L) : -INFINITY;
            const int tok = col / G, hh = col % G;
            const size_t hq = (size_t)d.kv_head * G + hh;
            if (d.partial_row < 0) {
                *reinterpret_cast<uint2*>(out + ((size_t)(d.out_row + tok) * Hq + hq) * D + dd) =
                    make_uint2(pack_bf16x2(a.x * inv, a.y * inv), pack_bf16x2(a.z * inv, a.w * inv));
                if (lse != nullptr && dd == 0) lse[(size_t)(d.out_row + tok) * Hq + hq] = lse2 * kLn2;
            } else {
                *reinterpret_cast<float4*>(p.partial_o + (((size_t)d.partial_row + tok) * G + hh) * D + dd) =
                    make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
                if (dd == 0) p.partial_lse[((size_t)d.partial_row + tok) * G + hh] = lse2;
            }
        }
        // the stage goes back to the producer (whose copies are writes of the asynchronous proxy) on
        // behalf of the eight consumer warps
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive_n(empty0 + 8 * d.stage, kWarps);
        if (d.partial_row < 0) continue;
        // ---- a chunk of a split unit: count it in; the CTA that completes the unit merges it
        __threadfence();      // this warp's partial rows are visible device-wide before the count moves
        __syncwarp();
        int last = 0;
        if (lane == 0) last = atomicAdd(p.unit_arrivals + d.unit, 1) == d.n_chunks - 1;
        if (__shfl_sync(0xffffffffu, last, 0) && !post(d)) break;
    }
}

// The merge warp's loop: LSE = log sum_c exp(LSE_c), O = sum_c exp(LSE_c - LSE) O_c over the chunks
// of a completed split unit, in chunk order.  All chunks are read back from memory (this CTA's own
// included), so the result does not depend on which CTA finished the unit.
template <int D, int G>
__device__ __forceinline__ void merge_loop(const DevPlan& p, __nv_bfloat16* __restrict__ out,
                                           float* __restrict__ lse, const TileDesc* merge_req,
                                           uint32_t req0, uint32_t reqfree0, volatile int* abort_flag) {
    const int lane = threadIdx.x & 31;
    const int Hq = p.num_q_heads;
    // merges one unit; dry: everything but the stores (see below)
    auto merge_unit = [&](const TileDesc& d, bool dry) {
        const int ncols = d.ntok * G;
        // four consecutive values of one column per lane and position; up to four positions and four
        // chunks per pass, all requested together: a unit of up to four chunks and 512 values costs
        // one round trip to L2
        for (int e0 = 4 * lane; e0 < ncols * D; e0 += 512) {
            float4 acc[4];
            float mx[4], wsum[4];
            size_t prow0[4], hh[4];
            int dd[4];
            bool on[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + 128 * u;
                on[u] = e < ncols * D;
                const int col = on[u] ? e / D : 0;
                dd[u] = e % D;
                hh[u] = (size_t)(col % G);
                prow0[u] = (size_t)d.partial_base + col / G;       // chunk c -> prow0 + c * ntok
                acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                mx[u] = -INFINITY;
                wsum[u] = 0.f;
            }
            for (int c0 = 0; c0 < d.n_chunks; c0 += 4) {
                float l2[4][4];
                float4 v[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        l2[u][i] = -INFINITY;
                        v[u][i] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (on[u] && c0 + i < d.n_chunks) {
                            const size_t r = (prow0[u] + (size_t)(c0 + i) * d.ntok) * G + hh[u];
                            l2[u][i] = __ldcg(p.partial_lse + r);
                            v[u][i] = __ldcg(reinterpret_cast<const float4*>(p.partial_o + r * D + dd[u]));
                        }
                    }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float pm = mx[u];
#pragma unroll
                    for (int i = 0; i < 4; ++i) pm = fmaxf(pm, l2[u][i]);
                    const float rescale = pm == -INFINITY ? 1.f : fast_exp2(mx[u] - pm);      // first pass: exp2(-inf) = 0
                    mx[u] = pm;
                    wsum[u] *= rescale;
                    acc[u].x *= rescale; acc[u].y *= rescale; acc[u].z *= rescale; acc[u].w *= rescale;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float w = l2[u][i] == -INFINITY ? 0.f : fast_exp2(l2[u][i] - mx[u]);   // -inf: no visible key there
                        wsum[u] += w;
                        if (w != 0.f) {
                            acc[u].x = fmaf(w, v[u][i].x, acc[u].x); acc[u].y = fmaf(w, v[u][i].y, acc[u].y);
                            acc[u].z = fmaf(w, v[u][i].z, acc[u].z); acc[u].w = fmaf(w, v[u][i].w, acc[u].w);
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (!on[u]) continue;
                const int col = (e0 + 128 * u) / D, tok = col / G;
                const float inv = 1.f / wsum[u];
                const size_t hq = (size_t)d.kv_head * G + hh[u];
                if (dry) continue;
                *reinterpret_cast<uint2*>(out + ((size_t)(d.out_row + tok) * Hq + hq) * D + dd[u]) =
                    make_uint2(pack_bf16x2(acc[u].x * inv, acc[u].y * inv), pack_bf16x2(acc[u].z * inv, acc[u].w * inv));
                if (lse != nullptr && dd[u] == 0)
                    lse[(size_t)(d.out_row + tok) * Hq + hq] = (mx[u] + log2f(wsum[u])) * kLn2;
            }
        }
    };
    // This code runs once or twice per CTA, at the very end of the step, where every microsecond of
    // cold instruction fetches shows; so it is run once up front, on partial rows that hold nothing
    // yet and with the stores left out, while the CTA waits for its first pages anyway.
    if (p.num_split_units > 0) {
        TileDesc warm{};
        warm.ntok = 1;
        warm.n_chunks = 1;
        warm.partial_base = 0;
        merge_unit(warm, true);
    }
    pdl_wait();
    for (int k = 0;; ++k) {
        const int j = k % kMergeReqs;
        if (!mbar_wait(req0 + 8 * j, (uint32_t)(k / kMergeReqs) & 1u, abort_flag, p.status, 5)) break;
        const TileDesc d = merge_req[j];
        __syncwarp();
        if (lane == 0) mbar_arrive(reqfree0 + 8 * j);
        if (d.flags & kFlagEnd) break;
        __threadfence();      // the chunks' rows were written before their counts moved: visible now
        merge_unit(d, false);
        if (lane == 0) atomicExch(p.unit_arrivals + d.unit, 0);      // ready for the next launch of this plan
        if (lane == 0) trace_add(7, 1);
    }
    if (lane == 0) trace_mark(3);
}

// The whole kernel body: warps 0-7 consume, warp 8 produces, warps 9 and 10 are the epilogue and the
// merge warp, any further warps of the CTA return at once (the fused kernel has twelve).
template <int D, int GT, bool APPEND>
__device__ __forceinline__ void decode_body(const DevPlan& p, const CUtensorMap* kv_map,
                                            const __nv_bfloat16* __restrict__ q,
                                            __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                            int S, uint8_t* smem, const AppendSrc& app) {
    using Geo = Geometry<D>;
    constexpr int G = GT;
    static_assert(G <= kCols && kCols % G == 0, "heads per kv head must divide the column count");
    uint8_t* stage_base = smem;                                        // 1024-byte aligned
    uint8_t* q_base = stage_base + (size_t)S * Geo::STAGE_BYTES;
    TileDesc* desc = (TileDesc*)(q_base + (size_t)S * Geo::Q_BYTES);
    TileDesc* handoff = desc + S;                // what the epilogue warp needs to know about a finished item
    TileDesc* merge_req = handoff + kHandoffs;   // completed split units on their way to the merge warp
    NextItem* next_item = (NextItem*)(merge_req + kMergeReqs);
    uint64_t* bars = (uint64_t*)(next_item + 1);   // full[S], empty[S], done[kHandoffs], req, reqfree, next full, free
    volatile int* abort_flag = (volatile int*)(bars + 2 * S + kHandoffs + 2 * kMergeReqs + 2);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + S), done0 = smem_u32(bars + 2 * S);
    const uint32_t req0 = done0 + 8 * kHandoffs, reqfree0 = req0 + 8 * kMergeReqs;
    const uint32_t next_full = reqfree0 + 8 * kMergeReqs, next_free = next_full + 8;

    if (threadIdx.x == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(kv_map));
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kWarps);
        }
        for (int h = 0; h < kHandoffs; ++h) mbar_init(done0 + 8 * h, kWarps);
        for (int j = 0; j < 2 * kMergeReqs + 2; ++j) mbar_init(req0 + 8 * j, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int Hq = p.num_q_heads;

    if (warp > kFetchWarp) return;      // further warps of the CTA have nothing to do
    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer warp
        // Its own first item (if the planner gave it one) comes inline in the CTA's header with its
        // first 32 page ids, so that the first copies leave after one round trip to memory; every
        // later item arrives from the fetch warp through shared memory, ready to issue.
        struct PItem { int kv0, kv_end, q_row0, ntok, kv_limit0, kv_head, partial_row, page0, unit, n_chunks, partial_base; };
        int n = 0;
        const int32_t* head = p.cta_heads + (size_t)blockIdx.x * kHeadWords;
        const int i0 = head[2], i1 = head[3];
        auto unpack = [](const int32_t* w) {
            PItem r;
            r.kv0 = w[0]; r.kv_end = w[1]; r.q_row0 = w[2]; r.ntok = w[3];
            r.kv_limit0 = w[4]; r.kv_head = w[5]; r.partial_row = w[6]; r.page0 = w[7];
            r.unit = w[8]; r.n_chunks = w[9]; r.partial_base = w[10];
            return r;
        };
        auto load_pages = [&](const PItem& it, int first_page) {
            const int npg = (it.kv_end - it.kv0 + kPage - 1) / kPage;
            const int idx = first_page + lane;
            return idx < npg ? __ldg(p.page_indices + it.page0 + idx) : 0;
        };
        constexpr int kPagesPerTile = kTileTok / kPage;       // 8
        constexpr int kGroupTiles = 32 / kPagesPerTile;       // 4
        bool ok = true;
        int taken = 0;
        int pages_cur = 0;
        // next item from the fetch warp (kv_end == 0: none); also sets pages_cur to its first 32 page ids
        auto take = [&]() {
            PItem r{0, 0, 0, 0, 0, 0, -1, 0, 0, 1, -1};
            ok = mbar_wait(next_full, (uint32_t)taken & 1u, abort_flag, p.status, 6);
            if (ok) {
                r = unpack(next_item->work);
                pages_cur = next_item->pages[lane];
                __syncwarp();
                if (lane == 0) mbar_arrive(next_free);
                ++taken;
            }
            return r;
        };
        PItem cur{0, 0, 0, 0, 0, 0, -1, 0, 0, 1, -1};
        if (i0 < i1 && !APPEND) {      // (with the append fused in, every item passes the fetch warp)
            cur = unpack(head + kHeadWorkCuda);
            pages_cur = head[kHeadPagesCuda + lane];
        }
        // The plan was uploaded before the kernel in front of this one started, so all of the above
        // overlaps that kernel's tail; the pool, Q and the queue are touched only from here on.
        pdl_wait();
        if (cur.kv_end == 0) cur = take();      // a CTA that came from span tiles starts on the queue
        while (cur.kv_end > 0 && ok) {
            const int ntiles = (cur.kv_end - cur.kv0 + kTileTok - 1) / kTileTok;
            for (int t0 = 0; t0 < ntiles && ok; t0 += kGroupTiles) {
                int pages_nxt = 0;
                const int t1 = min(t0 + kGroupTiles, ntiles);
                for (int t = t0; t < t1; ++t, ++n) {
                    const int s = n % S;
                    const uint32_t ph = (uint32_t)(n / S) & 1u;
                    ok = mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag, p.status, 1);
                    if (!ok) break;
                    const int base = cur.kv0 + t * kTileTok;
                    const int rows = min(kTileTok, cur.kv_end - base);
                    const int npages = (rows + kPage - 1) / kPage;
                    const bool first = t == 0;
                    if (lane == 0) {
                        TileDesc d;
                        d.flags = (first ? kFlagFirst : 0) | (t == ntiles - 1 ? kFlagLast : 0);
                        d.rows = rows;
                        d.lim0 = cur.kv_limit0 - base;
                        d.ntok = cur.ntok;
                        d.out_row = cur.q_row0;
                        d.kv_head = cur.kv_head;
                        d.partial_row = cur.partial_row;
                        d.unit = cur.unit;
                        d.n_chunks = cur.n_chunks;
                        d.partial_base = cur.partial_base;
                        d.stage = s;
                        d.pad = 0;
                        desc[s] = d;
                        mbar_arrive_expect_tx(full0 + 8 * s,
                                              (uint32_t)(npages * Geo::PAGE_BYTES + (first ? cur.ntok * G * D * 2 : 0)));
                    }
                    __syncwarp();
                    int page = __shfl_sync(0xffffffffu, pages_cur,
                                           (t - t0) * kPagesPerTile + (lane < kPagesPerTile ? lane : 0));
                    // checked build only: a bad id is replaced by page 0 (the copy must happen: the stage counts its bytes)
                    if (lane < npages && !page_ok(page, p.num_pages, p.status, kStatusBadPageWarp)) page = 0;
                    if (lane == 0) { if (n == 0) trace_mark(2); trace_add(6, 1); if (first) trace_add(5, 1); }
                    if (lane < npages)
                        tma_page_kv(smem_u32(stage_base + (size_t)s * Geo::STAGE_BYTES + (size_t)lane * Geo::PAGE_BYTES),
                                    kv_map, cur.kv_head, page, full0 + 8 * s);
                    // the unit's query rows: G * d contiguous values per token, columns in (token, head) order
                    if (first && lane >= 16 && lane - 16 < cur.ntok) {
                        const int tok = lane - 16;
                        const __nv_bfloat16* src = q + ((size_t)(cur.q_row0 + tok) * Hq + (size_t)cur.kv_head * G) * D;
                        bulk_g2s(smem_u32(q_base + (size_t)s * Geo::Q_BYTES + (size_t)tok * G * D * 2), src,
                                 G * D * 2, full0 + 8 * s);
                    }
                    // page ids of the next group of stages are requested after this group's first stage has left
                    if (t == t0 && t0 + kGroupTiles < ntiles) pages_nxt = load_pages(cur, (t0 + kGroupTiles) * kPagesPerTile);
                }
                pages_cur = pages_nxt;
            }
            if (ok) cur = take();
        }
        if (ok) {
            const int s = n % S;
            const uint32_t ph = (uint32_t)(n / S) & 1u;
            if (mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag, p.status, 1)) {
                if (lane == 0) {
                    desc[s].flags = kFlagEnd;
                    mbar_arrive(full0 + 8 * s);
                }
            }
        } else {
            // aborted: let the copies already issued land before the CTA's shared memory goes away
            const long long t0 = clock64();
            for (int k = max(0, n - S); k < n; ++k)
                while (!mbar_try_wait(full0 + 8 * (k % S), (uint32_t)(k / S) & 1u) &&
                       clock64() - t0 < kWaitCycles) {}
        }
        // the last CTA to leave the queue puts its counters back to zero for the next launch
        if (p.queue_count > 0 && lane == 0 && atomicAdd(p.counters + 1, 1) == (int)gridDim.x - 1) {
            atomicExch(p.counters, 0);
            atomicExch(p.counters + 1, 0);
        }
        return;
    }

    if (warp == kEpilogueWarp) {
        epilogue_loop<D, G>(p, out, lse, stage_base, handoff, merge_req, empty0, done0, req0, reqfree0, abort_flag);
        return;
    }
    if (warp == kMergeWarp) {
        merge_loop<D, G>(p, out, lse, merge_req, req0, reqfree0, abort_flag);
        return;
    }
    if (warp == kFetchWarp) {
        // ------------------------------------------------------------------ fetch warp
        // Runs one item ahead of the producer: the CTA's own items (beyond the first, which the producer
        // reads from the header itself), then the queue, one atomic add per chunk.  A chunk is claimed
        // only when the producer has taken the one before it, so a CTA never holds more than one chunk
        // it has not started.
        const int32_t* head = p.cta_heads + (size_t)blockIdx.x * kHeadWords;
        const int i1 = head[3];
        int own = head[2] < i1 && !APPEND ? head[2] + 1 : head[2];
        pdl_wait();      // the queue's counter belongs to the launch in front until that has completed
        for (int j = 0;; ++j) {
            if (j > 0 && !mbar_wait(next_free, (uint32_t)(j - 1) & 1u, abort_flag, p.status, 7)) break;
            int idx = -1;
            if (own < i1) {
                idx = own++;
            } else if (p.queue_count > 0) {
                int k = 0;
                if (lane == 0) k = atomicAdd(p.counters, 1);
                k = __shfl_sync(0xffffffffu, k, 0);
                if (k < p.queue_count) idx = p.queue_first + k;
            }
            int w = 0, pg = 0;
            if (idx >= 0) {
                const int32_t* rec = reinterpret_cast<const int32_t*>(p.works + idx);
                if (lane < 12) w = __ldg(rec + lane);
                const int kv0 = __shfl_sync(0xffffffffu, w, 0), kv_end = __shfl_sync(0xffffffffu, w, 1);
                const int page0 = __shfl_sync(0xffffffffu, w, 7);
                if (lane < (kv_end - kv0 + kPage - 1) / kPage) pg = __ldg(p.page_indices + page0 + lane);
                if constexpr (APPEND) {
                    // asynclm_step: the new K/V rows this item reads go into their page slots now; the
                    // producer's copies (asynchronous proxy) come after the hand-off below
                    Work rec;
                    rec.kv0 = kv0; rec.kv_end = kv_end; rec.page0 = page0;
                    rec.q_row0 = __shfl_sync(0xffffffffu, w, 2);
                    rec.kv_limit0 = __shfl_sync(0xffffffffu, w, 4);
                    rec.kv_head = __shfl_sync(0xffffffffu, w, 5);
                    rec.q_seq0 = __shfl_sync(0xffffffffu, w, 11);
                    append_rows_of_item(p, app, rec, lane);
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                }
            }
            if (lane < 12) next_item->work[lane] = w;
            next_item->pages[lane] = pg;
            __syncwarp();
            if (lane == 0) mbar_arrive(next_full);
            if (idx < 0) break;
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    pdl_wait();
    const int g = lane >> 2, t4 = lane & 3;      // fragment coordinates
    const float qscale = p.sm_scale * kLog2e;
    // ldmatrix row addresses inside a page slot, without the per-step piece index:
    //   K (plain): matrices (keys 0-7, k 0-7), (keys 8-15, k 0-7), (keys 0-7, k 8-15), (keys 8-15, k 8-15)
    //   V (transposed): (keys 0-7, d 0-7), (keys 0-7, d 8-15), (keys 8-15, d 0-7), (keys 8-15, d 8-15)
    const int k_key = (lane & 7) + ((lane >> 3) & 1) * 8, k_piece = lane >> 4;
    const int v_key = (lane & 7) + (lane >> 4) * 8, v_piece = (lane >> 3) & 1;
    const uint32_t k_row = (uint32_t)k_key * 128u, v_row = (uint32_t)Geo::BLOCK_BYTES + (uint32_t)v_key * 128u;
    const uint32_t k_swz = (uint32_t)(k_key & 7), v_swz = (uint32_t)(v_key & 7);

    uint32_t qb[Geo::KSTEPS][2];      // B fragments of Q^T: column g, values 16 ks + 2 t4 (+1) and + 8
    float o[Geo::KSTEPS][4];          // O^T: rows d = 16 i + g (+8), columns 2 t4, 2 t4 + 1
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;      // of columns 2 t4 and 2 t4 + 1
    int item_count = 0;

    for (int n = 0;; ++n) {
        const int s = n % S;
        const uint32_t ph = (uint32_t)(n / S) & 1u;
        if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.status, 2)) break;
        const TileDesc d = desc[s];
        if (d.flags & kFlagEnd) {
            // tell the epilogue warp that nothing follows
            if (threadIdx.x == 0) { trace_mark(4); handoff[item_count % kHandoffs].flags = kFlagEnd; }
            __syncwarp();
            if (lane == 0) mbar_arrive(done0 + 8 * (item_count % kHandoffs));
            break;
        }
        uint8_t* stage = stage_base + (size_t)s * Geo::STAGE_BYTES;
        if (d.flags & kFlagFirst) {
            const uint8_t* qs = q_base + (size_t)s * Geo::Q_BYTES;
            const bool col_valid = g < d.ntok * G;
#pragma unroll
            for (int ks = 0; ks < Geo::KSTEPS; ++ks) {
                const uint32_t* src = reinterpret_cast<const uint32_t*>(qs + ((size_t)g * D + ks * 16 + t4 * 2) * 2);
                qb[ks][0] = col_valid ? src[0] : 0u;
                qb[ks][1] = col_valid ? src[4] : 0u;
#pragma unroll
                for (int e = 0; e < 4; ++e) o[ks][e] = 0.f;
            }
            m0 = m1 = -INFINITY;
            l0 = l1 = 0.f;
        }
        const int key0 = warp * kPage;                    // this warp's page inside the stage
        if (key0 < d.rows) {
            const uint32_t page_smem = smem_u32(stage) + (uint32_t)warp * Geo::PAGE_BYTES;
            const int valid = d.rows - key0;              // slots of the page that hold keys of the sequence
            if (valid < kPage) {
                // Slots past the sequence's end hold whatever was in the page before: their scores are
                // masked below, but 0 * NaN would still poison P V, so their V rows are cleared.
                for (int r = valid + (lane >> 4); r < kPage; r += 2)
#pragma unroll
                    for (int h = 0; h < Geo::HALVES; ++h)
                        if ((lane & 15) < 8)
                            *reinterpret_cast<uint4*>(stage + (size_t)warp * Geo::PAGE_BYTES + Geo::BLOCK_BYTES + h * 2048 +
                                                      r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                __syncwarp();
            }
            // ---- S^T = K Q^T, two accumulators so that the MMAs are not one dependent chain
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < Geo::KSTEPS; ++ks) {
                const int piece = 2 * ks + k_piece;       // 16-byte piece of the row: half piece / 8
                uint32_t a[4];
                ldsm_x4(page_smem + (uint32_t)(piece >> 3) * 2048u + k_row + ((((uint32_t)piece & 7u) ^ k_swz) << 4), a);
                if (ks & 1) mma_bf16(sb, a, qb[ks][0], qb[ks][1]);
                else mma_bf16(sa, a, qb[ks][0], qb[ks][1]);
            }
            float sc[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[e] = (sa[e] + sb[e]) * qscale;      // log2 domain
            // ---- mask: key key0 + g (+8) is visible to column c iff it lies below lim0 + token(c)
            if (d.lim0 < key0 + kPage) {
                const int lim_a = d.lim0 + (2 * t4) / G - key0, lim_b = d.lim0 + (2 * t4 + 1) / G - key0;
                if (g >= lim_a) sc[0] = -INFINITY;
                if (g >= lim_b) sc[1] = -INFINITY;
                if (g + 8 >= lim_a) sc[2] = -INFINITY;
                if (g + 8 >= lim_b) sc[3] = -INFINITY;
            }
            // ---- softmax against the lazily moved reference maxima of this thread's two columns
            float c0 = fmaxf(sc[0], sc[2]), c1 = fmaxf(sc[1], sc[3]);
            if (__any_sync(0xffffffffu, c0 > m0 + kRescaleThreshold || c1 > m1 + kRescaleThreshold)) {
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    c0 = fmaxf(c0, __shfl_xor_sync(0xffffffffu, c0, off));
                    c1 = fmaxf(c1, __shfl_xor_sync(0xffffffffu, c1, off));
                }
                const float n0 = fmaxf(m0, c0), n1 = fmaxf(m1, c1);
                const float f0 = n0 == -INFINITY ? 1.f : fast_exp2(m0 - n0);
                const float f1 = n1 == -INFINITY ? 1.f : fast_exp2(m1 - n1);
                m0 = n0; m1 = n1;
                l0 *= f0; l1 *= f1;
#pragma unroll
                for (int i = 0; i < Geo::KSTEPS; ++i) {
                    o[i][0] *= f0; o[i][1] *= f1; o[i][2] *= f0; o[i][3] *= f1;
                }
            }
            const float u0 = m0 == -INFINITY ? 0.f : m0, u1 = m1 == -INFINITY ? 0.f : m1;
            const float p0 = fast_exp2(sc[0] - u0), p1 = fast_exp2(sc[1] - u1);
            const float p2 = fast_exp2(sc[2] - u0), p3 = fast_exp2(sc[3] - u1);
            l0 += p0 + p2;
            l1 += p1 + p3;
            // P (keys x columns, bf16) -> P^T as the B operand: two 8x8 transposes in registers
            const uint32_t b0 = movmatrix_t(pack_bf16x2(p0, p1));
            const uint32_t b1 = movmatrix_t(pack_bf16x2(p2, p3));
            // ---- O^T += V^T P^T
#pragma unroll
            for (int i = 0; i < Geo::KSTEPS; ++i) {
                const int piece = 2 * i + v_piece;
                uint32_t a[4];
                ldsm_x4_t(page_smem + (uint32_t)(piece >> 3) * 2048u + v_row + ((((uint32_t)piece & 7u) ^ v_swz) << 4), a);
                mma_bf16(o[i], a, b0, b1);
            }
        }

        if (!(d.flags & kFlagLast)) {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);
            continue;
        }
        // ---- end of item: leave this warp's state in its own page slot of the stage (only this warp
        // read that slot) for the epilogue warp, and go on
        {
            float* st = reinterpret_cast<float*>(stage + (size_t)warp * Geo::PAGE_BYTES);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            __syncwarp();      // every lane is done reading the page before it is overwritten
#pragma unroll
            for (int i = 0; i < Geo::KSTEPS; ++i) {
                float* c = st + (size_t)(2 * t4) * Geo::O_STRIDE + 16 * i + g;
                c[0] = o[i][0];
                c[Geo::O_STRIDE] = o[i][1];
                c[8] = o[i][2];
                c[Geo::O_STRIDE + 8] = o[i][3];
            }
            if (g == 0) {
                float* ms = st + kCols * Geo::O_STRIDE;
                ms[2 * t4] = m0; ms[2 * t4 + 1] = m1;
                ms[kCols + 2 * t4] = l0; ms[kCols + 2 * t4 + 1] = l1;
            }
            const int h = item_count % kHandoffs;
            if (threadIdx.x == 0) handoff[h] = d;
            __syncwarp();
            if (lane == 0) mbar_arrive(done0 + 8 * h);
            ++item_count;
        }
    }
}

}  // namespace dec

}  // namespace asynclm
