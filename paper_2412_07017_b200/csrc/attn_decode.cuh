// CUDA-core attention for decode rows (and spans too short for the tensor-core path).
//
// Each new token attends to its sequence's whole cached context plus its own span up to itself
// (paper Section 3.2 / 5.3: interrupt tokens are appended to the context and processed in the next
// decoding step, next to the other sequences' one-token decodes).  This path is bound by HBM
// bandwidth: every K/V row is read once and used by the G query heads that share the kv head.
//
// Structure: one persistent CTA per SM walks the item list the planner gave it.  A producer warp
// streams the items' K/V pages (contiguous 16-token blocks) into a shared-memory ring with bulk
// asynchronous copies that complete on mbarriers, together with a small descriptor and the query
// rows of each item.  Twelve consumer warps each take 8 rows of a 96-row tile: fp32 dot products
// with packed two-wide FMAs, a select-free transposing shuffle reduction, softmax against a lazily
// updated reference maximum, and the P.V update; at the end of an item the warps' states are merged
// through shared memory and written either as final bf16 output or as an fp32 partial for the
// split-KV merge.  The path is bound by instruction latency rather than by any one pipe, so the
// warp count matters: registers are moved from the producer's warpgroup to the consumers
// (setmaxnreg) to keep twelve of them resident.
//
// Every wait is bounded: a wait that runs out sets the plan's device status word and a CTA-wide
// abort flag, after which all loops fall through and the kernel returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace asynclm {

namespace dec {

constexpr int kWarps = 12;                   // consumer warps (three warpgroups)
constexpr int kThreads = (kWarps + 4) * 32;  // + the producer's warpgroup (one working warp)
constexpr int kRowsPerWarp = 8;
// A warp works on at most 4 query heads (the accumulators of more do not fit its registers).  With
// 8 heads per kv head the warps split into two halves that take 4 heads each and share the K/V
// rows in shared memory: 6 row blocks x 2 head halves, 48-row tiles instead of 96.
__host__ __device__ constexpr int head_splits(int group) { return group > 4 ? group / 4 : 1; }
// Register budget: the CTA is launched with 512 x 128 registers; the producer's warpgroup gives
// most of its share back and the consumers take it: 384 x 160 + 128 x 24 = 64512 <= 65536.
constexpr int kRegsConsumer = 152, kRegsProducer = 56;
static_assert(kWarps * 32 * kRegsConsumer + 128 * kRegsProducer <= 65536, "register split");
constexpr float kRescaleThreshold = 16.f;    // log2 units a score may exceed the reference max by
constexpr long long kWaitCycles = 2000000000ll;

constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagEnd = 4;

struct TileDesc {
    int32_t flags;
    int32_t rows;         // valid rows in this tile
    int32_t out_row;      // global token row of the item
    int32_t kv_head;
    int32_t partial_row;  // -1: final output
    int32_t pad[3];
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

// One tiled TMA copy fetches the K block and the V block of a (page, kv head): the pool is described
// to the TMA unit as a 5-D tensor [pages][2][Hkv][16][d] and the box spans (d, 16, 1, 2, 1), i.e. two
// separate 16 x d blocks of global memory that land back to back in shared memory.  (A bulk/TMA
// copy costs about 70 cycles plus 1 cycle per 107 bytes on this part, so halving the number of
// copies matters.)  No multicast.
__device__ __forceinline__ void tma_page_kv(uint32_t dst, const CUtensorMap* map, int kv_head, int page, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(0), "r"(0), "r"(kv_head), "r"(0), "r"(page), "r"(bar) : "memory");
}

__device__ __forceinline__ float2 unpack2(uint32_t w) { return make_float2(bf16_lo(w), bf16_hi(w)); }

// Transposing reduction over the LPR lanes that share a row.  Every lane starts with N values that
// must each be summed over the LPR lanes; each stage halves the number of values a lane keeps
// (while more than one is left) and adds the partner's copy of the kept half.  No selects are
// needed because a lane fills its slots in a lane-dependent order: slot k of lane `sub` holds the
// value with true index k ^ mask(sub), mask(sub) = sub * N / LPR (or sub >> log2(LPR / N) when
// N < LPR), so at every stage all lanes keep the lower half of their slots and send the upper
// half.  Afterwards slot f of lane `sub` holds the complete sum of true index
// sub * (N / LPR) + f (or sub >> log2(LPR / N) when N < LPR, duplicated over neighbouring lanes).
template <int N, int OFF, int NMAX>
__device__ __forceinline__ void transpose_reduce(float (&v)[NMAX]) {
    if constexpr (OFF >= 1) {
        if constexpr (N > 1) {
#pragma unroll
            for (int j = 0; j < N / 2; ++j)
                v[j] += __shfl_xor_sync(0xffffffffu, v[j + N / 2], OFF);
            transpose_reduce<N / 2, OFF / 2, NMAX>(v);
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], OFF);
            transpose_reduce<1, OFF / 2, NMAX>(v);
        }
    }
}

constexpr int ilog2(int x) { return x <= 1 ? 0 : 1 + ilog2(x / 2); }

template <int D, int G, int HS = 1>     // G: heads per warp, HS: head halves per CTA
struct Geometry {
    static constexpr int LPR = D / 8;                 // lanes per row (16 bytes each)
    static constexpr int TPW = 32 / LPR;              // rows per warp-wide shared-memory load
    static constexpr int NR = kRowsPerWarp / TPW;     // rows per lane
    static constexpr int NV = NR * G;                 // partial dot products per lane
    static constexpr int NF = NV >= LPR ? NV / LPR : 1;              // finished scores per lane
    static constexpr int DUP_SHIFT = NV >= LPR ? 0 : ilog2(LPR / NV); // lanes holding duplicates
    static constexpr int PAGE_BYTES = kPage * D * 2;
    static constexpr int ROW_BLOCKS = kWarps / HS;
    static constexpr int TILE_TOK = ROW_BLOCKS * kRowsPerWarp;          // rows per ring stage: 96 or 48
    // a stage holds, page after page, the page's K block followed by its V block
    static constexpr int STAGE_BYTES = (TILE_TOK / kPage) * 2 * PAGE_BYTES;
    static constexpr int Q_BYTES = G * HS * D * 2;
    static constexpr int STAT_FLOATS = (kWarps * G + 7) / 8 * 8;         // max (or sum) array, padded to 32 bytes
    static constexpr int MERGE_FLOATS = 2 * STAT_FLOATS + kWarps * G * D;  // one merge buffer
    // A lane's slot (i, g) holds the partial score of true row i ^ xi and true head g ^ xg, with
    // (xi, xg) = (mask / G, mask % G) and mask as in transpose_reduce.  The finished score of a
    // lane's slot (i, g) sits in slot score_slot(i, g) of the lane whose index differs from its own
    // by score_xor(i, g).
    __host__ __device__ static constexpr int score_xor(int i, int g) {
        return NV >= LPR ? (i * G + g) / NF : (i * G + g) << DUP_SHIFT;
    }
    __host__ __device__ static constexpr int score_slot(int i, int g) { return NV >= LPR ? (i * G + g) % NF : 0; }
};

template <int D, int GT>
size_t smem_bytes(int stages) {
    using Geo = Geometry<D, GT / head_splits(GT), head_splits(GT)>;
    return (size_t)stages * (Geo::STAGE_BYTES + Geo::Q_BYTES + sizeof(TileDesc) + 16) +
           2 * Geo::MERGE_FLOATS * sizeof(float) + 3 * 8 + 16 + 1024;
}

// The whole kernel body.  FUSED: the CTA has just finished the tensor-core phase of the fused
// kernel, in which warps 0-7 held 168 registers, warps 8-11 held 80 and warps 12-15 held 24.
template <int D, int GT, bool FUSED>
__device__ __forceinline__ void decode_body(const DevPlan& p, const CUtensorMap* kv_map,
                                            const __nv_bfloat16* __restrict__ q,
                                            __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                            int S, uint8_t* smem) {
    constexpr int HS = head_splits(GT);     // head halves
    constexpr int G = GT / HS;              // query heads per warp
    using Geo = Geometry<D, G, HS>;
    constexpr int LPR = Geo::LPR, TPW = Geo::TPW, NR = Geo::NR, NV = Geo::NV, NF = Geo::NF;
    constexpr int RB = Geo::ROW_BLOCKS, kTileTok = Geo::TILE_TOK;
    uint8_t* stage_base = smem;
    uint8_t* q_base = stage_base + (size_t)S * Geo::STAGE_BYTES;
    float* merge_base = (float*)(q_base + (size_t)S * Geo::Q_BYTES);
    TileDesc* desc = (TileDesc*)(merge_base + 2 * Geo::MERGE_FLOATS);
    uint64_t* bars = (uint64_t*)(desc + S);      // full[S], empty[S], merge[2]
    volatile int* abort_flag = (volatile int*)(bars + 2 * S + 2);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + S), mbar0 = smem_u32(bars + 2 * S);

    if (threadIdx.x == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(kv_map));
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kWarps);
        }
        mbar_init(mbar0, kWarps);
        mbar_init(mbar0 + 8, kWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int Hq = p.num_q_heads;

    if (warp >= kWarps) {
        if constexpr (!FUSED) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsProducer));
        else asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsProducer));      // idled with 24 so far
        if (warp > kWarps) return;      // the other warps of the producer's warpgroup have nothing to do
        // ------------------------------------------------------------------ producer warp
        // The page ids of the next 32 pages (8 tiles) and the descriptors of the next two items are
        // fetched ahead of use, so that no global-load latency sits between two tiles.
        struct PItem { int kv0, kv_end, q_row0, kv_head, partial_row, page0; };
        int n = 0;
        // the CTA's header gives its item range, its first item and that item's first 32 page ids in
        // one round trip to memory
        const int32_t* head = p.cta_heads + (size_t)blockIdx.x * kHeadWords;
        const int i0 = head[2], i1 = head[3];
        auto load_item = [&](int ii) {
            PItem r{0, 0, 0, 0, -1, 0};
            if (ii < i1) {
                const int4* src = ii == i0 ? reinterpret_cast<const int4*>(head + kHeadWorkCuda)
                                           : reinterpret_cast<const int4*>(p.works + ii);
                const int4 a = __ldg(src), b = __ldg(src + 1);
                r.kv0 = a.x; r.kv_end = a.y; r.q_row0 = a.z;
                r.kv_head = b.y; r.partial_row = b.z; r.page0 = b.w;
            }
            return r;
        };
        auto load_pages = [&](const PItem& it, int first_page) {
            const int npg = (it.kv_end - it.kv0 + kPage - 1) / kPage;
            const int idx = first_page + lane;
            return idx < npg ? __ldg(p.page_indices + it.page0 + idx) : 0;
        };
        constexpr int kPagesPerTile = kTileTok / kPage;
        constexpr int kGroupTiles = 32 / kPagesPerTile;
        bool ok = true;
        PItem cur = load_item(i0), nxt = load_item(i0 + 1);
        int pages_cur = head[kHeadPagesCuda + lane];
        // The plan was uploaded before the kernel in front of this one started, so all of the above
        // overlaps that kernel's tail; the pool and Q are read only from here on.
        pdl_wait();
        for (int ii = i0; cur.kv_end > 0 && ok; ++ii) {
            const PItem after = load_item(ii + 2);
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
                        d.out_row = cur.q_row0;
                        d.kv_head = cur.kv_head;
                        d.partial_row = cur.partial_row;
                        desc[s] = d;
                        mbar_arrive_expect_tx(full0 + 8 * s,
                                              (uint32_t)(npages * 2 * Geo::PAGE_BYTES + (first ? Geo::Q_BYTES : 0)));
                    }
                    __syncwarp();
                    const int64_t page = __shfl_sync(0xffffffffu, pages_cur,
                                                     (t - t0) * kPagesPerTile + (lane < kPagesPerTile ? lane : 0));
                    if (lane < npages)
                        tma_page_kv(smem_u32(stage_base + (size_t)s * Geo::STAGE_BYTES + lane * 2 * Geo::PAGE_BYTES),
                                    kv_map, cur.kv_head, (int)page, full0 + 8 * s);
                    if (first && lane == 31) {
                        const __nv_bfloat16* src = q + ((size_t)cur.q_row0 * Hq + (size_t)cur.kv_head * GT) * D;
                        bulk_g2s(smem_u32(q_base + (size_t)s * Geo::Q_BYTES), src, Geo::Q_BYTES, full0 + 8 * s);
                    }
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
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    pdl_wait();      // outputs may be written only after the kernel in front has completed
    if constexpr (FUSED) {
        if (warp < 8) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsConsumer));
        else asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsConsumer));
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsConsumer));
    }
    const int sub = lane % LPR;
    const int grp = lane / LPR;
    const int my_row = (sub >> 2) * TPW + grp;   // row (within the warp's 8) of this lane's scores
    const int mask = NV >= LPR ? sub * NF : sub >> Geo::DUP_SHIFT;
    const int xi = mask / G;                     // this lane's slot i holds true row i ^ xi
    const int xg = mask % G;                     // and its slot g holds true head g ^ xg
    const float qscale = p.sm_scale * kLog2e;

    float2 q2[G][4];
    float2 o2[G][4];
    float m_ref[G];
    float m_own[NF], l_own[NF];
    int item_count = 0;
    int32_t cur_out_row = 0, cur_kv_head = 0, cur_partial = -1;

    for (int n = 0;; ++n) {
        const int s = n % S;
        const uint32_t ph = (uint32_t)(n / S) & 1u;
        if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.status, 2)) break;
        const TileDesc d = desc[s];
        if (d.flags & kFlagEnd) break;
        if (d.flags & kFlagFirst) {
            const uint8_t* qs = q_base + (size_t)s * Geo::Q_BYTES;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint4 w = *reinterpret_cast<const uint4*>(qs + ((size_t)((warp / RB) * G + (g ^ xg)) * D + sub * 8) * 2);
                q2[g][0] = unpack2(w.x); q2[g][1] = unpack2(w.y);
                q2[g][2] = unpack2(w.z); q2[g][3] = unpack2(w.w);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    q2[g][j].x *= qscale; q2[g][j].y *= qscale;
                    o2[g][j] = make_float2(0.f, 0.f);
                }
                m_ref[g] = -INFINITY;
            }
#pragma unroll
            for (int f = 0; f < NF; ++f) { m_own[f] = -INFINITY; l_own[f] = 0.f; }
            cur_out_row = d.out_row; cur_kv_head = d.kv_head; cur_partial = d.partial_row;
        }
        const int rows = d.rows;
        const int blk = warp % RB;      // row block of the tile; warp / RB is the head half
        const bool active = blk * kRowsPerWarp < rows;
        uint4 kw[NR], vw[NR];
        if (active) {
            // the warp's 8 rows are one half of a page: [page][K 16 rows | V 16 rows]
            const uint8_t* ks = stage_base + (size_t)s * Geo::STAGE_BYTES + (size_t)(blk >> 1) * 2 * Geo::PAGE_BYTES +
                                (size_t)((blk & 1) * kRowsPerWarp) * (D * 2) + lane * 16;
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                kw[i] = *reinterpret_cast<const uint4*>(ks + (size_t)(i ^ xi) * TPW * D * 2);
                vw[i] = *reinterpret_cast<const uint4*>(ks + Geo::PAGE_BYTES + (size_t)(i ^ xi) * TPW * D * 2);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * s);

        if (active) {
            const bool tail = rows < (blk + 1) * kRowsPerWarp;
            if (tail) {
#pragma unroll
                for (int i = 0; i < NR; ++i)
                    if (blk * kRowsPerWarp + (i ^ xi) * TPW + grp >= rows) {
                        kw[i] = make_uint4(0, 0, 0, 0);
                        vw[i] = make_uint4(0, 0, 0, 0);
                    }
            }
            // scores: partial dot products over this lane's 8 elements, then reduce over the row's lanes
            float v[NV];
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                const float2 k0 = unpack2(kw[i].x), k1 = unpack2(kw[i].y), k2 = unpack2(kw[i].z), k3 = unpack2(kw[i].w);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float2 a = __fmul2_rn(q2[g][0], k0);
                    a = __ffma2_rn(q2[g][1], k1, a);
                    a = __ffma2_rn(q2[g][2], k2, a);
                    a = __ffma2_rn(q2[g][3], k3, a);
                    v[i * G + g] = a.x + a.y;
                }
            }
            transpose_reduce<NV, LPR / 2, NV>(v);
            float sc[NF];
#pragma unroll
            for (int f = 0; f < NF; ++f) sc[f] = v[f];
            if (tail && blk * kRowsPerWarp + my_row >= rows) {
#pragma unroll
                for (int f = 0; f < NF; ++f) sc[f] = -INFINITY;
            }
            bool need = false;
#pragma unroll
            for (int f = 0; f < NF; ++f) need |= sc[f] > m_own[f] + kRescaleThreshold;
            if (__any_sync(0xffffffffu, need)) {
                // move the reference maximum: per head, over this warp's rows of the tile
                float mn[NF];
#pragma unroll
                for (int f = 0; f < NF; ++f) {
                    float t = sc[f];
                    t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 4));
                    t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 8));
                    t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, 16));
                    mn[f] = fmaxf(m_own[f], t);
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float mg = __shfl_xor_sync(0xffffffffu, mn[Geo::score_slot(0, g)], Geo::score_xor(0, g));
                    const float scale = fast_exp2(m_ref[g] - mg);
                    m_ref[g] = mg;
                    const float2 s2 = make_float2(scale, scale);
#pragma unroll
                    for (int j = 0; j < 4; ++j) o2[g][j] = __fmul2_rn(o2[g][j], s2);
                }
#pragma unroll
                for (int f = 0; f < NF; ++f) {
                    l_own[f] *= fast_exp2(m_own[f] - mn[f]);
                    m_own[f] = mn[f];
                }
            }
            float pr[NF];
#pragma unroll
            for (int f = 0; f < NF; ++f) {
                pr[f] = fast_exp2(sc[f] - m_own[f]);
                l_own[f] += pr[f];
            }
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                const float2 v0 = unpack2(vw[i].x), v1 = unpack2(vw[i].y), v2 = unpack2(vw[i].z), v3 = unpack2(vw[i].w);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float pg = __shfl_xor_sync(0xffffffffu, pr[Geo::score_slot(i, g)], Geo::score_xor(i, g));
                    const float2 pp = make_float2(pg, pg);
                    o2[g][0] = __ffma2_rn(pp, v0, o2[g][0]);
                    o2[g][1] = __ffma2_rn(pp, v1, o2[g][1]);
                    o2[g][2] = __ffma2_rn(pp, v2, o2[g][2]);
                    o2[g][3] = __ffma2_rn(pp, v3, o2[g][3]);
                }
            }
        }

        if (d.flags & kFlagLast) {
            // ---- end of item: merge the warps' states and write the result
            float* mm = merge_base + (size_t)(item_count & 1) * Geo::MERGE_FLOATS;   // [warp][G] max
            float* ml = mm + Geo::STAT_FLOATS;                                    // [warp][G] sum
            float* mo = ml + Geo::STAT_FLOATS;                                    // [warp][G][D]
#pragma unroll
            for (int f = 0; f < NF; ++f) {
                l_own[f] += __shfl_xor_sync(0xffffffffu, l_own[f], 4);
                l_own[f] += __shfl_xor_sync(0xffffffffu, l_own[f], 8);
                l_own[f] += __shfl_xor_sync(0xffffffffu, l_own[f], 16);
            }
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                for (int g = 0; g < G; ++g)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        o2[g][j].x += __shfl_xor_sync(0xffffffffu, o2[g][j].x, off);
                        o2[g][j].y += __shfl_xor_sync(0xffffffffu, o2[g][j].y, off);
                    }
            if (grp == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float4* dst = reinterpret_cast<float4*>(mo + ((size_t)warp * G + (g ^ xg)) * D + sub * 8);
                    dst[0] = make_float4(o2[g][0].x, o2[g][0].y, o2[g][1].x, o2[g][1].y);
                    dst[1] = make_float4(o2[g][2].x, o2[g][2].y, o2[g][3].x, o2[g][3].y);
                }
                if ((sub >> 2) == 0) {
#pragma unroll
                    for (int f = 0; f < NF; ++f) {
                        const int k = NV >= LPR ? sub * NF + f : sub >> Geo::DUP_SHIFT;
                        const int g = k % G;
                        mm[warp * G + g] = m_own[f];
                        ml[warp * G + g] = l_own[f];
                    }
                }
            }
            __syncwarp();
            const int buf = item_count & 1;
            const uint32_t mb = mbar0 + 8 * buf;
            if (lane == 0) mbar_arrive(mb);
            // barrier `buf` serves every second item; its phase flips once per use
            if (!mbar_wait(mb, (uint32_t)(item_count >> 1) & 1u, abort_flag, p.status, 3)) break;
            ++item_count;
            const int tid = threadIdx.x;
            for (int e = 2 * tid; e < GT * D; e += 2 * kWarps * 32) {
                const int gfull = e / D, dd = e % D;
                const int g = gfull % G, w0 = (gfull / G) * RB;      // the RB warps that hold this head
                float M = -INFINITY;
#pragma unroll
                for (int r = 0; r < RB; ++r) M = fmaxf(M, mm[(w0 + r) * G + g]);
                float L = 0.f, a0 = 0.f, a1 = 0.f;
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const int w = w0 + r;
                    const float wgt = fast_exp2(mm[w * G + g] - M);
                    L = fmaf(ml[w * G + g], wgt, L);
                    const float2 ov = *reinterpret_cast<const float2*>(mo + ((size_t)w * G + g) * D + dd);
                    a0 = fmaf(ov.x, wgt, a0);
                    a1 = fmaf(ov.y, wgt, a1);
                }
                const float inv = 1.f / L;
                const size_t hq = (size_t)cur_kv_head * GT + gfull;
                if (cur_partial < 0) {
                    *reinterpret_cast<uint32_t*>(out + ((size_t)cur_out_row * Hq + hq) * D + dd) =
                        pack_bf16x2(a0 * inv, a1 * inv);
                    if (lse != nullptr && dd == 0)
                        lse[(size_t)cur_out_row * Hq + hq] = (M + log2f(L)) * kLn2;
                } else {
                    *reinterpret_cast<float2*>(p.partial_o + ((size_t)cur_partial * GT + gfull) * D + dd) =
                        make_float2(a0 * inv, a1 * inv);
                    if (dd == 0) p.partial_lse[(size_t)cur_partial * GT + gfull] = M + log2f(L);
                }
            }
        }
    }
}

}  // namespace dec

}  // namespace asynclm
