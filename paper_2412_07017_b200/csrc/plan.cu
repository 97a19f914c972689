// Host planner: validates one step's batch, tiles it into (unit, KV chunk) work items, balances the
// items over persistent CTAs and uploads the packed plan with one asynchronous copy.
//
// The step being planned is the "next decoding step" after the interrupt manager has appended its
// queued interrupt tokens (paper Section 5.3): q_len 1 = decode, > 1 = interrupt span, 0 = a
// sequence paused by a trap (Section 3.2).  All work here is integer work on the host.
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>
#include <cstring>
#include <vector>

#include "asynclm.h"
#include "plan_internal.h"

namespace asynclm {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int resolve_num_sms(const asynclm_plan_options* opts, bool need_device, int* out) {
    if (opts && opts->num_sms > 0) { *out = opts->num_sms; return ASYNCLM_OK; }
    if (!need_device) { *out = 148; return ASYNCLM_OK; }
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ASYNCLM_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return ASYNCLM_ERR_CUDA;
    *out = n;
    return ASYNCLM_OK;
}

static int check_shape(const asynclm_shape* s) {
    if (!s) return ASYNCLM_ERR_INVALID_ARG;
    if (s->num_q_heads <= 0 || s->num_kv_heads <= 0 || s->num_pages < 0 || s->reserved != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    if (s->num_q_heads % s->num_kv_heads != 0) return ASYNCLM_ERR_UNSUPPORTED_SHAPE;
    const int g = s->num_q_heads / s->num_kv_heads;
    if (!(g == 1 || g == 2 || g == 4 || g == 8)) return ASYNCLM_ERR_UNSUPPORTED_SHAPE;
    if (!(s->head_dim == 64 || s->head_dim == 128)) return ASYNCLM_ERR_UNSUPPORTED_SHAPE;
    if (s->page_size != kPage) return ASYNCLM_ERR_UNSUPPORTED_SHAPE;
    return ASYNCLM_OK;
}

// Tokens of a span that one tensor-core work item covers: two row tiles of 128 (token, head) rows.
int tensor_tile_tokens(int group) { return 256 / group; }

// Rows (G * q_len) from which a (sequence, kv head) goes to the span body (tcgen05).  Below it the
// warp body reads the keys once per 8 (token, head) columns, which costs less than a span item's
// start-up; decode rows (G rows) always stay on the warp body, which runs at the memory rate for
// every supported G.
static int default_tensor_min_rows(int) { return 32; }

// Sizes of the sections of the packed blob (identical offsets on host and device).
struct BlobLayout {
    size_t off_q_indptr, off_kv_len, off_page_indptr, off_page_indices, off_row_seq, off_row_slot, off_units,
        off_items, off_works, off_heads, off_cta_cuda, off_cta_tensor, off_split, off_merge, off_status,
        off_arrivals, blob_bytes;
};

static BlobLayout layout_blob(int batch, int total_q, int64_t total_pages, int64_t n_units,
                              int64_t n_items, int ctas_cuda, int ctas_tensor, int64_t n_split,
                              int64_t n_merge_blocks) {
    BlobLayout L{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    L.off_status = take(256);
    L.off_q_indptr = take(sizeof(int32_t) * (size_t)(batch + 1));
    L.off_kv_len = take(sizeof(int32_t) * (size_t)std::max(batch, 1));
    L.off_page_indptr = take(sizeof(int32_t) * (size_t)(batch + 1));
    L.off_page_indices = take(sizeof(int32_t) * (size_t)std::max<int64_t>(total_pages, 1));
    L.off_row_seq = take(sizeof(int32_t) * (size_t)std::max(total_q, 1));
    L.off_row_slot = take(sizeof(int64_t) * (size_t)std::max(total_q, 1));
    L.off_units = take(sizeof(Unit) * (size_t)std::max<int64_t>(n_units, 1));
    L.off_items = take(sizeof(Item) * (size_t)std::max<int64_t>(n_items, 1));
    L.off_works = take(sizeof(Work) * (size_t)std::max<int64_t>(n_items, 1));
    L.off_heads = take(sizeof(int32_t) * kHeadWords * (size_t)std::max(ctas_cuda, ctas_tensor));
    L.off_cta_cuda = take(sizeof(int32_t) * (size_t)(ctas_cuda + 1));
    L.off_cta_tensor = take(sizeof(int32_t) * (size_t)(ctas_tensor + 1));
    L.off_split = take(sizeof(int32_t) * (size_t)std::max<int64_t>(n_split, 1));
    L.off_merge = take(sizeof(int32_t) * (size_t)std::max<int64_t>(n_merge_blocks, 1));
    L.off_arrivals = take(sizeof(int32_t) * (size_t)std::max<int64_t>(n_units, 1));
    L.blob_bytes = o;
    return L;
}

static size_t partial_bytes(int64_t rows, int group, int head_dim) {
    return align_up((size_t)rows * (size_t)group * (size_t)head_dim * sizeof(float), 256) +
           align_up((size_t)rows * (size_t)group * sizeof(float), 256);
}

// Warp-body units: a sixth of the work is cut into short chunks for the end of the queue, about
// kTailChunksPerCta per CTA and never shorter than kMinChunkTiles tiles (see deal_dynamic).
constexpr int kTailChunksPerCta = 2;
constexpr int kMinChunkTiles = 4;
// Tokens of one warp-body unit: its MMAs have 8 (token, head) columns.
static int warp_unit_tokens(int group) { return 8 / group; }

// Upper bounds on what the automatic policy produces.  Warp body: the short chunks are at least
// (all tiles) / (12 CTAs) long, so even a single unit that holds all the work yields at most 12 per
// CTA; a long piece is at least two fifths of a CTA's share.  Span body: a unit is cut only where it
// is larger than a CTA's share.
static int64_t auto_item_bound(int64_t units, int ctas) { return 2 * units + (int64_t)20 * ctas; }
static int64_t auto_partial_row_bound(int ctas, int group) {
    return (int64_t)20 * ctas * warp_unit_tokens(group) + (int64_t)3 * ctas * tensor_tile_tokens(group);
}

}  // namespace asynclm

using namespace asynclm;

extern "C" int asynclm_plan_workspace_size(const asynclm_shape* shape,
                                           const asynclm_plan_options* opts, int32_t max_batch,
                                           int32_t max_total_q, int64_t max_total_pages,
                                           size_t* host_bytes, size_t* device_bytes) {
    int rc = check_shape(shape);
    if (rc != ASYNCLM_OK) return rc;
    if (max_batch < 0 || max_total_q < 0 || max_total_pages < 0 || !host_bytes || !device_bytes)
        return ASYNCLM_ERR_INVALID_ARG;
    int n_sms = 0;
    if (resolve_num_sms(opts, true, &n_sms) != ASYNCLM_OK) n_sms = 160;
    const int G = shape->num_q_heads / shape->num_kv_heads;
    const int ctas_cuda = n_sms * kCudaSlotsPerSm;
    const int ctas_tensor = n_sms;
    const int64_t max_units = (int64_t)max_total_q * shape->num_kv_heads;
    int64_t max_items, max_partial_rows;
    if (opts && opts->kv_chunk_tokens > 0) {
        // fixed chunk length: every unit may be cut into ceil(n/chunk) pieces
        const int64_t per_unit = (max_total_pages * kPage) / opts->kv_chunk_tokens + 1;
        max_items = max_units * per_unit;
        max_partial_rows = max_items;   // ntok tokens per unit are already counted in max_units
    } else {
        max_items = auto_item_bound(max_units, ctas_cuda);
        max_partial_rows = auto_partial_row_bound(ctas_cuda, G);      // only cut units hold partial rows
    }
    BlobLayout L = layout_blob(max_batch, max_total_q, max_total_pages, max_units, max_items,
                               ctas_cuda, ctas_tensor, max_units,
                               (int64_t)max_total_q * shape->num_q_heads / 4 + max_units);
    *host_bytes = align_up(sizeof(asynclm_plan_s), 256) + L.blob_bytes +
                  align_up(sizeof(int32_t) * (size_t)std::max<int64_t>(max_items, 1), 256);
    *device_bytes = L.blob_bytes + partial_bytes(max_partial_rows, G, shape->head_dim);
    return ASYNCLM_OK;
}

namespace {

struct UnitBuild {
    Unit u;
    int path;
    int64_t n_keys;   // keys visible to the unit's last token
};

// Cuts the units of one path into items and deals them to `n_ctas` persistent CTAs.
// fixed_chunk > 0: equal chunks of that many tokens, then a contiguous equal-cost partition of the
// item sequence.  Otherwise: the concatenated tile sequence of all units is cut into n_ctas nearly
// equal contiguous ranges (a unit is split only where a range boundary falls inside it).
void cut_and_deal(const std::vector<int>& unit_ids, std::vector<UnitBuild>& units, int fixed_chunk,
                  int n_ctas, int item_overhead_tiles, std::vector<Item>& items,
                  std::vector<int32_t>& cta_indptr, std::vector<int32_t>& item_cta) {
    const size_t first_item = items.size();
    cta_indptr.assign((size_t)n_ctas + 1, (int32_t)first_item);
    if (unit_ids.empty() || n_ctas <= 0) return;
    auto tiles_of = [](int64_t tokens) { return (tokens + kKvTile - 1) / kKvTile; };
    if (fixed_chunk > 0) {
        for (int id : unit_ids) {
            UnitBuild& ub = units[id];
            int c = 0;
            for (int64_t k0 = 0; k0 < ub.n_keys; k0 += fixed_chunk, ++c) {
                Item it{id, (int32_t)k0, (int32_t)std::min<int64_t>(ub.n_keys, k0 + fixed_chunk), c};
                items.push_back(it);
            }
            ub.u.n_chunks = c;
        }
        int64_t total = 0;
        for (size_t i = first_item; i < items.size(); ++i)
            total += item_overhead_tiles + tiles_of(items[i].kv1 - items[i].kv0);
        // contiguous partition: an item goes to the CTA in whose share of the total its midpoint falls
        int64_t cum = 0;
        for (size_t i = first_item; i < items.size(); ++i) {
            const int64_t c = item_overhead_tiles + tiles_of(items[i].kv1 - items[i].kv0);
            const int64_t cta = std::min<int64_t>(n_ctas - 1, ((2 * cum + c) * n_ctas) / (2 * total));
            item_cta.push_back((int32_t)cta);
            cum += c;
        }
    } else {
        int64_t total_tiles = 0;
        for (int id : unit_ids) total_tiles += tiles_of(units[id].n_keys);
        const int64_t total_cost =
            total_tiles + (int64_t)item_overhead_tiles * ((int64_t)unit_ids.size() + n_ctas);
        const int64_t quota = std::max<int64_t>(1 + item_overhead_tiles,
                                                (total_cost + n_ctas - 1) / n_ctas);
        int cta = 0;
        int64_t budget = quota;
        for (int id : unit_ids) {
            UnitBuild& ub = units[id];
            int64_t tiles_left = tiles_of(ub.n_keys);
            int64_t k0 = 0;
            int c = 0;
            while (tiles_left > 0) {
                if (budget <= item_overhead_tiles && cta + 1 < n_ctas) {
                    ++cta;
                    budget = quota;
                }
                int64_t take = cta + 1 < n_ctas
                                   ? std::min<int64_t>(tiles_left, std::max<int64_t>(1, budget - item_overhead_tiles))
                                   : tiles_left;
                const int64_t k1 = std::min<int64_t>(ub.n_keys, k0 + take * kKvTile);
                items.push_back(Item{id, (int32_t)k0, (int32_t)k1, c});
                item_cta.push_back(cta);
                budget -= item_overhead_tiles + take;
                tiles_left -= take;
                k0 = k1;
                ++c;
            }
            ub.u.n_chunks = c;
        }
    }
    // items were emitted in CTA order; build the CSR
    std::vector<int32_t> count((size_t)n_ctas, 0);
    for (size_t i = first_item; i < items.size(); ++i) count[(size_t)item_cta[i]]++;
    int32_t at = (int32_t)first_item;
    for (int k = 0; k < n_ctas; ++k) {
        cta_indptr[(size_t)k] = at;
        at += count[(size_t)k];
    }
    cta_indptr[(size_t)n_ctas] = at;
}


// Measured costs of the attention kernels on B200, in nanoseconds, used only to size the span CTAs.
struct PathCost {
    int gran;            // tokens per tile of the path (cuts fall on multiples of it)
    int64_t tile_ns;     // one tile in steady state
    int64_t item_ns;     // starting and finishing an item (pipeline fill and drain, merge, write)
    int64_t phase_ns;    // first item of the path on a CTA (descriptor chain, first loads)
};
// Span body: a KV tile of 128 keys against one row tile, an item, the body's start on a CTA.
constexpr PathCost kTensorCost{128, 1170, 8000, 11800};
constexpr int64_t kTensorDualTileNs = 2435;   // a KV tile of an item with two row tiles (more than 128 rows)
// When every unit runs on the span body all SMs stream K/V tiles at once and the tile time is set by
// the memory system (64 KB per tile and SM); the producers run ahead across item boundaries.
constexpr PathCost kTensorOnlyCost{128, 1543, 8000, 2400};
constexpr int64_t kTensorOnlyDualTileNs = 3126;
// Warp body: 64 KB per 128-key tile.  It is bound by memory, so its tile time depends on how many SMs
// stream at once: 1.45 us when all 148 do, 1.05 us (62 KB/us, about what one SM can stream) when
// half of them run span tiles, which draw little bandwidth.  The model takes the latter figure.
constexpr PathCost kWarpCost{128, 1050, 400, 2000};
// No step ends before its bytes have crossed the memory bus: K/V pages stream at about 6 bytes per
// nanosecond on this access pattern (4 KB runs through a shuffled page table), after about 3 us in
// which the CTAs start.  Without this floor the model would spread the span units over so many CTAs
// that too few were left streaming to keep the memory busy (one SM streams 60-75 KB/us at most).
// Each (sequence, kv head) counts once: the row tiles of a long span re-read it, mostly from L2.
constexpr int64_t kDramBytesPerUs = 6000000;
// A span CTA that finishes early joins the queue; one that finishes late delays the whole step, and the
// span body slows down by up to 15 % when the warp-body CTAs saturate the memory.  So the span CTAs
// are filled to the load limit divided by this margin (in 1/64).
constexpr int64_t kSpanMargin64 = 72;
// Share (in 1/64) of the queue that the CTAs without span work must be able to stream by themselves.
constexpr int64_t kStreamShare64 = 58;
constexpr int64_t kStartNs = 3000;

// Default policy for the fused kernel.
//   Span units (tensor-core body) are compute-heavy and predictable: they are packed whole onto as few
// persistent CTAs as the load limit allows (largest first, each into the fullest CTA that still has
// room; a unit larger than a CTA's share is cut into equal pieces), so that most of them write final
// bf16 rows instead of fp32 partial rows.
//   Warp-body units (decode rows, short spans) are bandwidth-bound, and how fast a CTA streams depends
// on what the other SMs are doing, which no static cost predicts.  They are cut into chunks of a few
// tiles, sorted by length (longest first), and handed out at run time: the CTAs without span work
// start on one chunk each, every other chunk waits in a queue from which a CTA that runs out of work
// (a span CTA included) takes the next one with one atomic add.  Partial results are indexed by chunk
// and merged in chunk order, so the output does not depend on which CTA ran what.
//   The load limit is the smallest one under which the span units fit and the room left on all CTAs
// covers the modelled time of the queue; it is found by bisection.
void deal_dynamic(std::vector<int>& ids_tensor, const std::vector<int>& ids_warp,
                  std::vector<UnitBuild>& units, int group, int64_t kv_bytes, int n_ctas, std::vector<Item>& items,
                  std::vector<int32_t>& cta_indptr_warp, std::vector<int32_t>& cta_indptr_tensor,
                  std::vector<int32_t>& item_cta, int32_t* queue_first, int32_t* queue_count) {
    struct Piece { Item it; int32_t cta; };
    const bool tensor_only = ids_warp.empty();
    const PathCost tc = tensor_only ? kTensorOnlyCost : kTensorCost;
    const int64_t dual_tile_ns = tensor_only ? kTensorOnlyDualTileNs : kTensorDualTileNs;
    auto tiles_of = [](int64_t keys, int gran) { return (keys + gran - 1) / gran; };

    // ---- warp-body work as the model sees it (the chunks are cut below, once the number of CTAs
    // that start on the queue is known)
    int64_t warp_tiles = 0;
    for (int id : ids_warp) warp_tiles += tiles_of(units[id].n_keys, kWarpCost.gran);
    const int64_t warp_ns = warp_tiles * kWarpCost.tile_ns + (int64_t)ids_warp.size() * 2 * kWarpCost.item_ns;

    // ---- span units with two row tiles that would not fit a CTA whole are divided by rows into two
    // units of one row tile each (same CTA-time in total, and the second reader of the keys finds most
    // of them in L2) rather than by keys, which would cost fp32 partial rows and a merge.  The limit
    // used for the decision is the lower bound of the one found below.
    {
        int64_t work = warp_ns;
        for (int id : ids_tensor)
            work += tc.item_ns + tiles_of(units[id].n_keys, tc.gran) * (units[id].u.ntok * group > 128 ? dual_tile_ns : tc.tile_ns);
        const int64_t limit0 = std::max(work / n_ctas, kStartNs + kv_bytes * 1000 / kDramBytesPerUs) * 64 / kSpanMargin64;
        const int half = 128 / group;      // tokens of one row tile
        const size_t n0 = ids_tensor.size();
        for (size_t i = 0; i < n0; ++i) {
            const int id = ids_tensor[i];
            UnitBuild& ub = units[(size_t)id];
            if (ub.u.ntok * group <= 128) continue;
            if (tc.phase_ns + tc.item_ns + tiles_of(ub.n_keys, tc.gran) * dual_tile_ns <= limit0) continue;
            UnitBuild second = ub;
            second.u.q_row0 += half;
            second.u.ntok -= half;
            second.u.kv_limit0 += half;
            ub.u.ntok = half;
            ub.n_keys = (int64_t)ub.u.kv_limit0 + ub.u.ntok - 1;
            ids_tensor.push_back((int)units.size());
            units.push_back(second);
        }
    }

    // ---- span units under a load limit
    std::vector<int> order(ids_tensor);
    std::vector<int64_t> tiles(units.size()), tns(units.size());
    for (int id : order) {
        tiles[(size_t)id] = tiles_of(units[id].n_keys, tc.gran);
        tns[(size_t)id] = units[id].u.ntok * group > 128 ? dual_tile_ns : tc.tile_ns;
    }
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) {
        return tiles[(size_t)x] * tns[(size_t)x] > tiles[(size_t)y] * tns[(size_t)y];
    });
    std::vector<int64_t> load((size_t)n_ctas);
    std::vector<Piece> pieces_out;
    int used = 0;
    // Packs the span units under `cap`; returns false if they do not fit or leave too little room for
    // the queue.  With emit == false only the verdict is computed (the bisection's probes).
    int64_t span_work = 0;      // all span items without the per-CTA start
    for (int id : order) span_work += tc.item_ns + tiles[(size_t)id] * tns[(size_t)id];
    auto fill = [&](int64_t limit, bool emit) {
        // CTAs that may hold span work: the others have to be able to stream most of the queue by
        // themselves (span CTAs draw little bandwidth, and one SM streams only so much)
        const int64_t stream_ctas = limit > kStartNs
            ? (warp_tiles * kWarpCost.tile_ns * kStreamShare64 / 64 + (limit - kStartNs) - 1) / (limit - kStartNs) : n_ctas;
        const int64_t span_ctas = ids_warp.empty() ? n_ctas : n_ctas - stream_ctas;
        if (!order.empty() && span_ctas < 1) return false;
        // what a span CTA may be given: the span work spread over those CTAs with some slack for the
        // packing, at most the load limit less the safety margin.  Spreading the spans thin costs little (a
        // span CTA that is done early joins the queue), filling span CTAs to the brim risks a late finish.
        const int64_t thin = order.empty() ? 0 : span_work / span_ctas * 5 / 4 + tc.phase_ns + tc.item_ns + dual_tile_ns;
        const int64_t cap = std::min(limit * 64 / kSpanMargin64, std::max(thin, 2 * (tc.phase_ns + tc.item_ns)));
        pieces_out.clear();
        std::fill(load.begin(), load.end(), (int64_t)0);
        used = 0;
        int64_t least = INT64_MAX;      // lower bound of the smallest load among the span CTAs
        bool fits = true;
        for (int id : order) {
            const int64_t t = tiles[(size_t)id], ns = tns[(size_t)id];
            const int64_t fresh_room = std::max<int64_t>(1, (cap - tc.phase_ns - tc.item_ns) / ns);
            const int64_t pieces = t <= fresh_room ? 1 : (t + fresh_room - 1) / fresh_room;
            int64_t k0 = 0;
            for (int64_t c = 0; c < pieces; ++c) {
                const int64_t take = pieces == 1 ? t : t / pieces + (c < t % pieces ? 1 : 0);
                const int64_t need = tc.item_ns + take * ns;
                int best = -1;
                if (least + need <= cap)            // otherwise no span CTA has room: skip the scan
                    for (int k = 0; k < used; ++k)
                        if (load[(size_t)k] + need <= cap && (best < 0 || load[(size_t)k] > load[(size_t)best])) best = k;
                if (best < 0) {
                    if (used < n_ctas) {
                        best = used++;
                        load[(size_t)best] = tc.phase_ns;
                    } else {
                        fits = false;
                        best = 0;
                        for (int k = 1; k < n_ctas; ++k) if (load[(size_t)k] < load[(size_t)best]) best = k;
                    }
                }
                if (!fits && !emit) return false;
                const int64_t k1 = std::min<int64_t>(units[id].n_keys, k0 + take * tc.gran);
                if (emit) pieces_out.push_back(Piece{Item{id, (int32_t)k0, (int32_t)k1, (int32_t)c}, (int32_t)best});
                load[(size_t)best] += need;
                least = std::min(least, load[(size_t)best]);
                k0 = k1;
            }
        }
        // room for the queue: what the span CTAs have left after restarting on the warp body, and the
        // whole limit on the others
        int64_t room = 0;
        for (int k = 0; k < n_ctas; ++k)
            room += std::max<int64_t>(0, limit - load[(size_t)k] - kWarpCost.phase_ns);
        return fits && used <= span_ctas && room >= warp_ns;
    };
    const int64_t total = warp_ns + span_work;
    const int64_t floor_ns = kStartNs + kv_bytes * 1000 / kDramBytesPerUs;
    int64_t lo = std::max<int64_t>(std::max<int64_t>(1, total / n_ctas), floor_ns);
    int64_t hi = lo + lo / 4 + tc.item_ns + tc.phase_ns + kWarpCost.phase_ns;
    while (!fill(hi, false)) { lo = hi; hi += hi / 2; }
    for (int iter = 0; iter < 24 && hi - lo > std::max<int64_t>(50, hi / 128); ++iter) {      // to 0.8 %
        const int64_t mid = (lo + hi) / 2;
        if (fill(mid, false)) hi = mid; else lo = mid;
    }
    fill(hi, true);
    std::stable_sort(pieces_out.begin(), pieces_out.end(), [](const Piece& x, const Piece& y) { return x.cta < y.cta; });

    // ---- warp-body chunks.  An item boundary costs time and a split unit costs partial rows and a
    // merge, so most of the work stays in long pieces: a few units, a sixth of all tiles, are cut into
    // short chunks that go to the END of the queue, where they even out the CTAs' finishing times;
    // every other unit stays whole unless it is longer than two fifths of the step, in which case it is
    // cut into equal pieces.  The queue holds the long pieces longest first, then the short chunks.
    std::vector<int> warp_order(ids_warp);
    std::stable_sort(warp_order.begin(), warp_order.end(),
                     [&](int x, int y) { return units[x].n_keys > units[y].n_keys; });
    std::vector<Item> chunks, tail;
    chunks.reserve(ids_warp.size() + (size_t)n_ctas * 4);
    const int64_t bulk_max = std::max<int64_t>(kMinChunkTiles, hi * 2 / 5 / kWarpCost.tile_ns);
    const int64_t tail_target = warp_tiles / 6;
    const int64_t tail_chunk = std::max<int64_t>(kMinChunkTiles, tail_target / ((int64_t)n_ctas * kTailChunksPerCta));
    // which units are cut short: first those of up to four chunks (their merge is one round trip to
    // L2), longest first; longer ones only if that does not give a sixth of the tiles
    std::vector<char> to_tail(units.size(), 0);
    int64_t tail_tiles = 0;
    for (int pass = 0; pass < 2 && tail_tiles < tail_target; ++pass)
        for (int id : warp_order) {
            const int64_t t = tiles_of(units[id].n_keys, kWarpCost.gran);
            if (tail_tiles >= tail_target) break;
            if (to_tail[(size_t)id] || t <= tail_chunk + tail_chunk / 2 || (pass == 0 && t > 4 * tail_chunk)) continue;
            to_tail[(size_t)id] = 1;
            tail_tiles += t;
        }
    for (int id : warp_order) {
        const int64_t t = tiles_of(units[id].n_keys, kWarpCost.gran);
        const bool short_chunks = to_tail[(size_t)id] != 0;
        const int64_t piece_max = short_chunks ? tail_chunk : bulk_max;
        const int64_t pieces = t <= piece_max + piece_max / 2 ? 1 : (t + piece_max - 1) / piece_max;
        int64_t k0 = 0;
        for (int64_t c = 0; c < pieces; ++c) {
            const int64_t take = t / pieces + (c < t % pieces ? 1 : 0);
            const int64_t k1 = std::min<int64_t>(units[id].n_keys, k0 + take * kWarpCost.gran);
            (short_chunks ? tail : chunks).push_back(Item{id, (int32_t)k0, (int32_t)k1, (int32_t)c});
            k0 = k1;
        }
        units[id].u.n_chunks = (int32_t)pieces;
    }
    auto longer = [](const Item& x, const Item& y) { return x.kv1 - x.kv0 > y.kv1 - y.kv0; };
    std::stable_sort(chunks.begin(), chunks.end(), longer);
    std::stable_sort(tail.begin(), tail.end(), longer);
    chunks.insert(chunks.end(), tail.begin(), tail.end());

    // ---- emit: warp-body items first (one start chunk for every CTA without span work, then the
    // queue), then the span items grouped by CTA
    cta_indptr_warp.assign((size_t)n_ctas + 1, 0);
    cta_indptr_tensor.assign((size_t)n_ctas + 1, 0);
    const int n_start = (int)std::min<size_t>(chunks.size(), (size_t)(n_ctas - used));
    for (size_t i = 0; i < chunks.size(); ++i) {
        items.push_back(chunks[i]);
        item_cta.push_back(i < (size_t)n_start ? used + (int32_t)i : -1);
    }
    for (int k = 0; k <= n_ctas; ++k)
        cta_indptr_warp[(size_t)k] = std::min(std::max(k - used, 0), n_start);
    *queue_first = n_start;
    *queue_count = (int32_t)chunks.size() - n_start;
    const int32_t first = (int32_t)items.size();
    std::vector<int32_t> count((size_t)n_ctas, 0);
    for (const Piece& pz : pieces_out) {
        items.push_back(pz.it);
        item_cta.push_back(pz.cta);
        count[(size_t)pz.cta]++;
        units[pz.it.unit].u.n_chunks = std::max(units[pz.it.unit].u.n_chunks, pz.it.chunk + 1);
    }
    int32_t at = first;
    for (int k = 0; k < n_ctas; ++k) {
        cta_indptr_tensor[(size_t)k] = at;
        at += count[(size_t)k];
    }
    cta_indptr_tensor[(size_t)n_ctas] = at;
}

}  // namespace

extern "C" int asynclm_plan(const asynclm_shape* shape, const asynclm_plan_options* opts,
                            const asynclm_batch* batch, void* host_ws, size_t host_bytes,
                            void* dev_ws, size_t dev_bytes, void* stream,
                            asynclm_plan_t** out_plan) {
    int rc = check_shape(shape);
    if (rc != ASYNCLM_OK) return rc;
    if (!batch || !host_ws || !out_plan || batch->batch < 0) return ASYNCLM_ERR_INVALID_ARG;
    if (((uintptr_t)host_ws & 15) != 0 || ((uintptr_t)dev_ws & 255) != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    const int B = batch->batch;
    if (B > 0 && (!batch->q_indptr || !batch->kv_len_before || !batch->page_indptr))
        return ASYNCLM_ERR_INVALID_ARG;
    if (opts && (opts->kv_chunk_tokens < 0 || opts->num_sms < 0 || opts->tensor_min_rows < 0))
        return ASYNCLM_ERR_INVALID_ARG;
    if (opts && opts->kv_chunk_tokens > 0 && opts->kv_chunk_tokens % 64 != 0)
        return ASYNCLM_ERR_INVALID_ARG;
    const bool host_only = dev_ws == nullptr;
    if (host_only && !(opts && opts->num_sms > 0)) return ASYNCLM_ERR_INVALID_ARG;

    int device = -1;
    if (!host_only) {
        if (cudaGetDevice(&device) != cudaSuccess) return ASYNCLM_ERR_CUDA;
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess)
            return ASYNCLM_ERR_CUDA;
        if (major != 10) return ASYNCLM_ERR_ARCH;
    }
    int n_sms = 0;
    rc = resolve_num_sms(opts, !host_only, &n_sms);
    if (rc != ASYNCLM_OK) return rc;

    const int Hkv = shape->num_kv_heads;
    const int G = shape->num_q_heads / Hkv;
    const int P = shape->page_size;

    // ---- validation -------------------------------------------------------------------------
    static const int32_t zero_indptr[1] = {0};
    const int32_t* q_indptr = B > 0 ? batch->q_indptr : zero_indptr;
    const int32_t* page_indptr = B > 0 ? batch->page_indptr : zero_indptr;
    if (q_indptr[0] != 0 || page_indptr[0] != 0) return ASYNCLM_ERR_INVALID_ARG;
    int64_t total_kv = 0;
    for (int b = 0; b < B; ++b) {
        const int64_t ql = (int64_t)q_indptr[b + 1] - q_indptr[b];
        const int64_t np = (int64_t)page_indptr[b + 1] - page_indptr[b];
        if (ql < 0 || np < 0 || batch->kv_len_before[b] < 0) return ASYNCLM_ERR_INVALID_ARG;
        const int64_t n = (int64_t)batch->kv_len_before[b] + ql;
        if (n > INT32_MAX - kKvTile) return ASYNCLM_ERR_INVALID_ARG;
        if (ql > 0) {
            if (np * P < n) return ASYNCLM_ERR_PAGE_TABLE;
            total_kv += n;
        }
    }
    const int T = q_indptr[B];
    const int64_t total_pages = page_indptr[B];
    if (total_pages > 0 && !batch->page_indices) return ASYNCLM_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b) {
        const int64_t ql = (int64_t)q_indptr[b + 1] - q_indptr[b];
        if (ql == 0) continue;   // paused sequences are not read or written: their ids are not checked
        const int64_t need = ((int64_t)batch->kv_len_before[b] + ql + P - 1) / P;
        for (int64_t j = 0; j < need; ++j) {
            const int32_t pg = batch->page_indices[page_indptr[b] + j];
            if (pg < 0 || pg >= shape->num_pages) return ASYNCLM_ERR_PAGE_TABLE;
        }
    }
    if (opts && (opts->flags & ASYNCLM_PLAN_REJECT_ALIASED_WRITES)) {
        std::vector<int32_t> written;
        for (int b = 0; b < B; ++b) {
            const int ql = q_indptr[b + 1] - q_indptr[b];
            if (ql == 0) continue;
            const int lo = batch->kv_len_before[b] / P;
            const int hi = (batch->kv_len_before[b] + ql - 1) / P;
            for (int j = lo; j <= hi; ++j) written.push_back(batch->page_indices[page_indptr[b] + j]);
        }
        std::sort(written.begin(), written.end());
        if (std::adjacent_find(written.begin(), written.end()) != written.end())
            return ASYNCLM_ERR_PAGE_TABLE;
    }

    // ---- units ------------------------------------------------------------------------------
    const bool tensor_ok = !(opts && (opts->flags & ASYNCLM_PLAN_NO_TENSOR_PATH)) &&
                           tensor_path_compiled(shape->head_dim);
    const int tensor_min_rows =
        (opts && opts->tensor_min_rows > 0) ? opts->tensor_min_rows : default_tensor_min_rows(G);
    const int TQ = tensor_tile_tokens(G);
    std::vector<UnitBuild> units;
    std::vector<int> ids_cuda, ids_tensor;
    for (int b = 0; b < B; ++b) {
        const int ql = q_indptr[b + 1] - q_indptr[b];
        if (ql == 0) continue;
        const int ctx = batch->kv_len_before[b];
        const bool tensor = tensor_ok && (int64_t)G * ql >= tensor_min_rows;
        const int step = tensor ? TQ : warp_unit_tokens(G);
        for (int h = 0; h < Hkv; ++h) {
            for (int t0 = 0; t0 < ql; t0 += step) {
                UnitBuild ub{};
                ub.u.seq = b;
                ub.u.kv_head = h;
                ub.u.q_row0 = q_indptr[b] + t0;
                ub.u.ntok = std::min(step, ql - t0);
                ub.u.kv_limit0 = ctx + t0 + 1;
                ub.u.n_chunks = 0;
                ub.u.partial_base = -1;
                ub.u.page_base = page_indptr[b];
                ub.path = tensor ? kPathTensor : kPathCuda;
                ub.n_keys = (int64_t)ub.u.kv_limit0 + ub.u.ntok - 1;
                (tensor ? ids_tensor : ids_cuda).push_back((int)units.size());
                units.push_back(ub);
            }
        }
    }

    // ---- items and CTA assignment --------------------------------------------------------------
    const int fixed_chunk = opts ? opts->kv_chunk_tokens : 0;
    const int ctas_cuda = n_sms * kCudaSlotsPerSm;
    const int ctas_tensor = n_sms;
    std::vector<Item> items;
    std::vector<int32_t> item_cta, cta_indptr_cuda, cta_indptr_tensor;
    int n_items_cuda = 0;
    int32_t queue_first = 0, queue_count = 0;
    if (fixed_chunk > 0 || ctas_cuda != ctas_tensor) {
        cut_and_deal(ids_cuda, units, fixed_chunk, ctas_cuda, kCudaItemOverheadTiles, items,
                     cta_indptr_cuda, item_cta);
        n_items_cuda = (int)items.size();
        cut_and_deal(ids_tensor, units, fixed_chunk, ctas_tensor, kTensorItemOverheadTiles, items,
                     cta_indptr_tensor, item_cta);
    } else {
        // bytes of K and V the step has to read, each (sequence, kv head) counted once
        const int64_t kv_bytes = total_kv * Hkv * 4 * shape->head_dim;
        deal_dynamic(ids_tensor, ids_cuda, units, G, kv_bytes, ctas_cuda, items, cta_indptr_cuda, cta_indptr_tensor, item_cta,
                     &queue_first, &queue_count);
        n_items_cuda = queue_first + queue_count;
    }
    const int n_items = (int)items.size();

    // ---- partial rows ------------------------------------------------------------------------
    std::vector<int32_t> split_units, merge_blocks;   // merge block: 4 (token, head) rows of a split unit
    int64_t partial_rows = 0;
    for (size_t i = 0; i < units.size(); ++i) {
        if (units[i].u.n_chunks > 1) {
            units[i].u.partial_base = (int32_t)partial_rows;
            partial_rows += (int64_t)units[i].u.n_chunks * units[i].u.ntok;
            split_units.push_back((int32_t)i);
            if (i >= (size_t)(INT32_MAX >> 6)) return ASYNCLM_ERR_WORKSPACE_TOO_SMALL;
            // split units of the warp body are merged inside the attention kernel; those of the span
            // body by the merge kernel
            if (units[i].path == kPathTensor)
                for (int rb = 0; rb * 4 < units[i].u.ntok * G; ++rb) merge_blocks.push_back((int32_t)((i << 6) | (size_t)rb));
            if (partial_rows > INT32_MAX / 2) return ASYNCLM_ERR_WORKSPACE_TOO_SMALL;
        }
    }

    const int n_split = (int)split_units.size();

    // ---- pack ---------------------------------------------------------------------------------
    BlobLayout L = layout_blob(B, T, total_pages, (int64_t)units.size(), n_items, ctas_cuda,
                               ctas_tensor, (int64_t)n_split, (int64_t)merge_blocks.size());
    const size_t plan_bytes = align_up(sizeof(asynclm_plan_s), 256);
    const size_t item_cta_bytes = align_up(sizeof(int32_t) * (size_t)std::max(n_items, 1), 256);
    const size_t host_need = plan_bytes + L.blob_bytes + item_cta_bytes;
    const size_t dev_need = L.blob_bytes + partial_bytes(partial_rows, G, shape->head_dim);
    if (host_bytes < host_need) return ASYNCLM_ERR_WORKSPACE_TOO_SMALL;
    if (!host_only && dev_bytes < dev_need) return ASYNCLM_ERR_WORKSPACE_TOO_SMALL;

    char* hb = (char*)host_ws + plan_bytes;
    std::memset(hb + L.off_status, 0, 256);
    std::memset(hb + L.off_arrivals, 0, sizeof(int32_t) * std::max<size_t>(units.size(), 1));
    if (B > 0) {
        std::memcpy(hb + L.off_q_indptr, q_indptr, sizeof(int32_t) * (size_t)(B + 1));
        std::memcpy(hb + L.off_kv_len, batch->kv_len_before, sizeof(int32_t) * (size_t)B);
        std::memcpy(hb + L.off_page_indptr, page_indptr, sizeof(int32_t) * (size_t)(B + 1));
    } else {
        std::memset(hb + L.off_q_indptr, 0, sizeof(int32_t));
        std::memset(hb + L.off_page_indptr, 0, sizeof(int32_t));
    }
    if (total_pages > 0)
        std::memcpy(hb + L.off_page_indices, batch->page_indices, sizeof(int32_t) * (size_t)total_pages);
    int32_t* row_seq = (int32_t*)(hb + L.off_row_seq);
    int64_t* row_slot = (int64_t*)(hb + L.off_row_slot);
    for (int b = 0; b < B; ++b)
        for (int r = q_indptr[b]; r < q_indptr[b + 1]; ++r) {
            row_seq[r] = b;
            const int pos = batch->kv_len_before[b] + (r - q_indptr[b]);
            row_slot[r] = (int64_t)batch->page_indices[page_indptr[b] + pos / P] * P + pos % P;
        }
    Unit* h_units = (Unit*)(hb + L.off_units);
    for (size_t i = 0; i < units.size(); ++i) h_units[i] = units[i].u;
    if (n_items > 0) std::memcpy(hb + L.off_items, items.data(), sizeof(Item) * (size_t)n_items);
    int32_t* h_heads = (int32_t*)(hb + L.off_heads);
    std::memset(h_heads, 0, sizeof(int32_t) * kHeadWords * (size_t)std::max(ctas_cuda, ctas_tensor));
    Work* h_works = (Work*)(hb + L.off_works);
    for (int i = 0; i < n_items; ++i) {
        const Item& it = items[(size_t)i];
        const Unit& u = units[(size_t)it.unit].u;
        Work w;
        w.kv0 = it.kv0;
        w.kv_end = std::min(it.kv1, u.kv_limit0 + u.ntok - 1);
        w.q_row0 = u.q_row0;
        w.ntok = u.ntok;
        w.kv_limit0 = u.kv_limit0;
        w.kv_head = u.kv_head;
        w.partial_row0 = u.partial_base < 0 ? -1 : u.partial_base + it.chunk * u.ntok;
        w.page0 = u.page_base + it.kv0 / kPage;
        w.unit = it.unit;
        w.n_chunks = u.n_chunks;
        w.partial_base = u.partial_base;
        w.q_seq0 = q_indptr[u.seq];
        h_works[i] = w;
    }
    for (int c = 0; c < std::max(ctas_cuda, ctas_tensor); ++c) {
        int32_t* h = h_heads + (size_t)c * kHeadWords;
        const int32_t range[4] = {c < ctas_tensor ? cta_indptr_tensor[(size_t)c] : 0,
                                  c < ctas_tensor ? cta_indptr_tensor[(size_t)c + 1] : 0,
                                  c < ctas_cuda ? cta_indptr_cuda[(size_t)c] : 0,
                                  c < ctas_cuda ? cta_indptr_cuda[(size_t)c + 1] : 0};
        std::memcpy(h, range, sizeof(range));
        for (int path = 0; path < 2; ++path) {
            const int first = range[2 * path], last = range[2 * path + 1];
            if (first >= last) continue;
            const Work& w = h_works[first];
            std::memcpy(h + (path == 0 ? kHeadWorkTensor : kHeadWorkCuda), &w, sizeof(Work));
            const int npg = (w.kv_end - w.kv0 + kPage - 1) / kPage;
            for (int k = 0; k < 32 && k < npg; ++k)
                h[(path == 0 ? kHeadPagesTensor : kHeadPagesCuda) + k] = batch->page_indices[w.page0 + k];
        }
    }
    std::memcpy(hb + L.off_cta_cuda, cta_indptr_cuda.data(), sizeof(int32_t) * (size_t)(ctas_cuda + 1));
    std::memcpy(hb + L.off_cta_tensor, cta_indptr_tensor.data(),
                sizeof(int32_t) * (size_t)(ctas_tensor + 1));
    if (n_split > 0) std::memcpy(hb + L.off_split, split_units.data(), sizeof(int32_t) * split_units.size());
    if (!merge_blocks.empty())
        std::memcpy(hb + L.off_merge, merge_blocks.data(), sizeof(int32_t) * merge_blocks.size());
    int32_t* h_item_cta = (int32_t*)(hb + L.blob_bytes);
    if (n_items > 0) std::memcpy(h_item_cta, item_cta.data(), sizeof(int32_t) * (size_t)n_items);

    asynclm_plan_s* plan = (asynclm_plan_s*)host_ws;
    std::memset(plan, 0, sizeof(*plan));
    plan->magic = kPlanMagic;
    plan->shape = *shape;
    plan->device = device;
    plan->host_only = host_only ? 1 : 0;
    plan->h_units = h_units;
    plan->h_items = (const Item*)(hb + L.off_items);
    plan->h_item_cta = h_item_cta;
    plan->h_kv_len_before = (const int32_t*)(hb + L.off_kv_len);
    plan->h_units_path_split = n_items_cuda;
    for (int b = 0; b < B; ++b) plan->max_q_len = std::max(plan->max_q_len, q_indptr[b + 1] - q_indptr[b]);

    char* db = (char*)dev_ws;
    DevPlan& d = plan->dev;
    auto dp = [&](size_t off) { return host_only ? nullptr : (void*)(db + off); };
    d.status = (int32_t*)dp(L.off_status);
    d.counters = (int32_t*)dp(L.off_status + 64);
    d.queue_first = queue_first;
    d.queue_count = queue_count;
    d.q_indptr = (const int32_t*)dp(L.off_q_indptr);
    d.kv_len_before = (const int32_t*)dp(L.off_kv_len);
    d.page_indptr = (const int32_t*)dp(L.off_page_indptr);
    d.page_indices = (const int32_t*)dp(L.off_page_indices);
    d.row_seq = (const int32_t*)dp(L.off_row_seq);
    d.row_slot = (const int64_t*)dp(L.off_row_slot);
    d.units = (const Unit*)dp(L.off_units);
    d.items = (const Item*)dp(L.off_items);
    d.works = (const Work*)dp(L.off_works);
    d.cta_heads = (const int32_t*)dp(L.off_heads);
    d.cta_indptr_cuda = (const int32_t*)dp(L.off_cta_cuda);
    d.cta_indptr_tensor = (const int32_t*)dp(L.off_cta_tensor);
    d.split_units = (const int32_t*)dp(L.off_split);
    d.merge_blocks = (const int32_t*)dp(L.off_merge);
    d.unit_arrivals = (int32_t*)dp(L.off_arrivals);
    d.partial_o = (float*)dp(L.blob_bytes);
    d.partial_lse = (float*)dp(L.blob_bytes + align_up((size_t)partial_rows * (size_t)G *
                                                           (size_t)shape->head_dim * sizeof(float), 256));
    d.batch = B;
    d.total_q = T;
    d.num_units = (int32_t)units.size();
    d.num_items = n_items;
    d.num_items_cuda = n_items_cuda;
    d.num_items_tensor = n_items - n_items_cuda;
    d.num_split_units = n_split;
    d.num_merge_blocks = (int32_t)merge_blocks.size();
    d.num_ctas_cuda = ctas_cuda;
    d.num_ctas_tensor = ctas_tensor;
    d.num_q_heads = shape->num_q_heads;
    d.num_kv_heads = Hkv;
    d.head_dim = shape->head_dim;
    d.group = G;
    d.num_pages = shape->num_pages;
    d.sm_scale = shape->sm_scale > 0.f ? shape->sm_scale : 1.0f / sqrtf((float)shape->head_dim);

    asynclm_plan_info& info = plan->info;
    info.total_q = T;
    info.num_units = d.num_units;
    info.num_items = n_items;
    info.num_split_units = d.num_split_units;
    info.partial_rows = (int32_t)partial_rows;
    int max_chunk = 0;
    for (const Item& it : items) max_chunk = std::max(max_chunk, it.kv1 - it.kv0);
    info.kv_chunk_tokens = fixed_chunk > 0 ? fixed_chunk : (d.num_split_units ? max_chunk : INT32_MAX);
    info.num_ctas_cuda = ctas_cuda;
    info.num_ctas_tensor = ctas_tensor;
    info.num_items_tensor = d.num_items_tensor;
    info.launches_append = T > 0 ? 1 : 0;
    // span tiles and decode rows share one fused launch when a step has both (head_dim 128)
    info.launches_attn = ((n_items_cuda > 0 || d.num_items_tensor > 0) ? 1 : 0) + (merge_blocks.empty() ? 0 : 1);
    info.num_sms = n_sms;
    info.total_kv_tokens = total_kv;
    info.device_bytes_used = dev_need;
    info.host_bytes_used = host_need;

    if (!host_only) {
        cudaError_t e = cudaMemcpyAsync(db, hb, L.blob_bytes, cudaMemcpyHostToDevice,
                                        (cudaStream_t)stream);
        if (e != cudaSuccess) return ASYNCLM_ERR_CUDA;
    }
    *out_plan = plan;
    return ASYNCLM_OK;
}

extern "C" int asynclm_plan_get_info(const asynclm_plan_t* plan, asynclm_plan_info* info) {
    if (!plan || !info || plan->magic != kPlanMagic) return ASYNCLM_ERR_INVALID_ARG;
    *info = plan->info;
    return ASYNCLM_OK;
}

extern "C" int asynclm_plan_get_items(const asynclm_plan_t* plan, asynclm_item_view* out,
                                      int32_t capacity) {
    if (!plan || plan->magic != kPlanMagic || capacity < 0 || (capacity > 0 && !out))
        return ASYNCLM_ERR_INVALID_ARG;
    const int n = plan->dev.num_items;
    for (int i = 0; i < n && i < capacity; ++i) {
        const Item& it = plan->h_items[i];
        const Unit& u = plan->h_units[it.unit];
        asynclm_item_view v;
        v.seq = u.seq;
        v.kv_head = u.kv_head;
        v.tok0 = u.kv_limit0 - 1 - plan->h_kv_len_before[u.seq];
        v.ntok = u.ntok;
        v.kv0 = it.kv0;
        v.kv1 = it.kv1;
        v.path = i < plan->h_units_path_split ? kPathCuda : kPathTensor;
        v.cta = plan->h_item_cta[i];
        out[i] = v;
    }
    return n;
}
