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

// Rows (G * q_len) from which a (sequence, kv head) goes to the tensor-core kernel.  Up to 4 heads per
// kv head a decode row stays on the CUDA-core kernel, which then runs near the memory rate, and spans
// of 32 rows and more take the tensor cores.  With 8 heads per kv head every KV byte feeds twice the
// arithmetic and the CUDA-core kernel is bound by its FMAs at half the memory rate (measured:
// 2.4 TB/s against 4.1 TB/s on the 64/8-head batch), so there the 8 rows of a decode token already
// count as wide enough.
static int default_tensor_min_rows(int group) { return group >= 8 ? 8 : 32; }

// Sizes of the sections of the packed blob (identical offsets on host and device).
struct BlobLayout {
    size_t off_q_indptr, off_kv_len, off_page_indptr, off_page_indices, off_row_seq, off_row_slot, off_units,
        off_items, off_works, off_heads, off_cta_cuda, off_cta_tensor, off_split, off_merge, off_status, blob_bytes;
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
    L.blob_bytes = o;
    return L;
}

static size_t partial_bytes(int64_t rows, int group, int head_dim) {
    return align_up((size_t)rows * (size_t)group * (size_t)head_dim * sizeof(float), 256) +
           align_up((size_t)rows * (size_t)group * sizeof(float), 256);
}

// Upper bound on the number of items the automatic policy produces: every unit yields one item
// plus at most one extra cut per persistent CTA.
static int64_t auto_item_bound(int64_t units, int ctas) { return units + ctas; }

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
        max_items = auto_item_bound(max_units, ctas_cuda + ctas_tensor);
        // only cut units hold partial rows: at most 2 pieces per cut, tensor_tile_tokens rows each
        max_partial_rows = (int64_t)2 * (ctas_cuda + ctas_tensor) * tensor_tile_tokens(G) +
                           (int64_t)2 * (ctas_cuda + ctas_tensor);
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


// Measured costs of the attention kernels on B200, in nanoseconds, used only to balance CTAs.
struct PathCost {
    int gran;            // tokens per tile of the path (cuts fall on multiples of it)
    int64_t tile_ns;     // one tile in steady state
    int64_t item_ns;     // starting and finishing an item (pipeline fill and drain, merge, write)
    int64_t phase_ns;    // first item of the path on a CTA (descriptor chain, first loads)
};
// (fitted to per-CTA phase times of the fused kernel on the Llama-3-8B-shaped mixed batch)
constexpr PathCost kTensorCost{128, 1170, 8000, 11800};
constexpr PathCost kCudaCost{128, 900, 1200, 2000};
constexpr int64_t kTensorDualTileNs = 2435;   // a KV tile of an item with two row tiles (more than 128 rows)
// When every unit runs on the tensor-core kernel all SMs stream K/V tiles at once and the tile time is
// set by the memory system (64 KB per tile and SM: 148 SMs at 37 KB/us are 5.5 TB/s); the producers
// run ahead across item boundaries.
constexpr PathCost kTensorOnlyCost{128, 1543, 8000, 2400};
constexpr int64_t kTensorOnlyDualTileNs = 3126;
// Units with fewer (token, head) rows than this are cut wherever a CTA is full (their partial rows are
// a few KB); wider span units are kept whole where they fit.
constexpr int kWholeUnitMinRows = 32;
// Decode units that a span CTA takes along on the tensor-core body at most (estimated from its room).
constexpr int64_t kMaxNarrowUnitsPerCta = 4;

// Default policy for the fused kernel, in which a persistent CTA runs its tensor-core items and then,
// if it has any, its CUDA-core items: units are weighted with the measured costs and dealt under a
// per-CTA load limit (see `fill` below), where decode rows placed on a CTA with span work normally
// become tensor-core items so that the CTA runs one body only; the smallest limit that fits is found
// by bisection, so that all CTAs finish together as far as the cost model holds.
void deal_jointly(const std::vector<int>& ids_tensor, const std::vector<int>& ids_cuda,
                  std::vector<UnitBuild>& units, int group, int n_ctas, std::vector<Item>& items,
                  std::vector<int32_t>& cta_indptr_cuda, std::vector<int32_t>& cta_indptr_tensor,
                  std::vector<int32_t>& item_cta) {
    struct Piece { Item it; int32_t cta; };
    std::vector<Piece> best[2];
    const std::vector<int>* ids[2] = {&ids_tensor, &ids_cuda};
    const bool tensor_only = ids_cuda.empty();
    PathCost cost[2] = {tensor_only ? kTensorOnlyCost : kTensorCost, kCudaCost};
    const int64_t dual_tile_ns = tensor_only ? kTensorOnlyDualTileNs : kTensorDualTileNs;
    // a narrow item (one decode token's rows) on the tensor-core body: tile and item cost
    const int64_t narrow_tile_ns = tensor_only ? kTensorOnlyCost.tile_ns : 1400;
    const int64_t narrow_item_ns = 2900;
    auto tile_ns = [&](int path, int id) {
        return path == 0 && units[id].u.ntok * group > 128 ? dual_tile_ns : cost[path].tile_ns;
    };
    // Lower bound of the makespan: all work, one start per unit, one phase start per CTA.
    int64_t total = 0;
    for (int path = 0; path < 2; ++path)
        for (int id : *ids[path])
            total += cost[path].item_ns + (units[id].n_keys + cost[path].gran - 1) / cost[path].gran * tile_ns(path, id);
    // Deal the work under a per-CTA load limit `cap`; returns false if it does not fit.
    //   Span units first, whole wherever possible (an unsplit unit writes final bf16 rows: no fp32
    // partial rows, no merge): largest first, each into the fullest span CTA that still has room for
    // it, else into a fresh CTA; a unit larger than a CTA's share is cut into equal pieces.
    //   Decode units then fill every CTA up to the limit in CTA order; a unit is cut only where a
    // CTA is full.
    //   With emit == false only the verdict is computed (the bisection's probes).
    std::vector<int> tensor_order, tensor_narrow;      // span units packed whole; narrow units that fill up CTAs
    for (int id : ids_tensor)
        (units[id].u.ntok * group >= kWholeUnitMinRows ? tensor_order : tensor_narrow).push_back(id);
    std::vector<int64_t> tiles_of(units.size()), tns_of(units.size());
    for (int path = 0; path < 2; ++path)
        for (int id : *ids[path]) {
            tiles_of[(size_t)id] = (units[id].n_keys + cost[path].gran - 1) / cost[path].gran;
            tns_of[(size_t)id] = tile_ns(path, id);
        }
    auto unit_tiles = [&](int, int id) { return tiles_of[(size_t)id]; };
    std::stable_sort(tensor_order.begin(), tensor_order.end(), [&](int x, int y) {
        return tiles_of[(size_t)x] * tns_of[(size_t)x] > tiles_of[(size_t)y] * tns_of[(size_t)y];
    });
    std::vector<int64_t> load((size_t)n_ctas);
    int64_t avg_unit_ns = 1;      // mean cost of a CUDA-core unit
    if (!ids_cuda.empty()) {
        int64_t sum = 0;
        for (int id : ids_cuda) sum += cost[1].item_ns + tiles_of[(size_t)id] * cost[1].tile_ns;
        avg_unit_ns = std::max<int64_t>(1, sum / (int64_t)ids_cuda.size());
    }
    auto fill = [&](int64_t cap, std::vector<Piece> (&out)[2], bool emit) {
        out[0].clear();
        out[1].clear();
        if (emit) {
            out[0].reserve(ids_tensor.size() + (size_t)n_ctas);
            out[1].reserve(ids_cuda.size() + (size_t)n_ctas);
        }
        bool fits = true;
        std::fill(load.begin(), load.end(), (int64_t)0);
        int used = 0;                                   // CTAs that hold span work: [0, used)
        int64_t least = INT64_MAX;                      // lower bound of the smallest load among them
        {
            const PathCost& pc = cost[0];
            // tiles a fresh CTA takes, for the two kinds of span tile
            const int64_t fresh_single = std::max<int64_t>(1, (cap - pc.phase_ns - pc.item_ns) / pc.tile_ns);
            const int64_t fresh_dual = std::max<int64_t>(1, (cap - pc.phase_ns - pc.item_ns) / dual_tile_ns);
            for (int id : tensor_order) {
                const int64_t tns = tns_of[(size_t)id];
                const int64_t tiles = unit_tiles(0, id);
                const int64_t fresh_room = tns == pc.tile_ns ? fresh_single : fresh_dual;
                const int64_t pieces = tiles <= fresh_room ? 1 : (tiles + fresh_room - 1) / fresh_room;
                int64_t k0 = 0;
                for (int64_t c = 0; c < pieces; ++c) {
                    const int64_t take = pieces == 1 ? tiles : tiles / pieces + (c < tiles % pieces ? 1 : 0);
                    const int64_t need = pc.item_ns + take * tns;
                    int best_cta = -1;
                    if (least + need <= cap)            // otherwise no span CTA has room: skip the scan
                        for (int k = 0; k < used; ++k)
                            if (load[(size_t)k] + need <= cap && (best_cta < 0 || load[(size_t)k] > load[(size_t)best_cta])) best_cta = k;
                    if (best_cta < 0) {
                        if (used < n_ctas) {
                            best_cta = used++;
                            load[(size_t)best_cta] = pc.phase_ns;
                        } else {
                            fits = false;
                            best_cta = 0;
                            for (int k = 1; k < n_ctas; ++k) if (load[(size_t)k] < load[(size_t)best_cta]) best_cta = k;
                        }
                    }
                    const int64_t k1 = std::min<int64_t>(units[id].n_keys, k0 + take * pc.gran);
                    if (emit) out[0].push_back(Piece{Item{id, (int32_t)k0, (int32_t)k1, (int32_t)c}, (int32_t)best_cta});
                    else if (!fits) return false;
                    load[(size_t)best_cta] += need;
                    least = std::min(least, load[(size_t)best_cta]);
                    k0 = k1;
                }
            }
        }
        // Line fill: the units of `list` in order, each CTA up to the limit; a unit is cut only where a
        // CTA is full.  CTAs below `started` already hold tensor-core work.  A CUDA-core unit (one decode
        // token) that lands on such a CTA runs there as a narrow tensor-core item: the CTA then never
        // re-splits its registers and restarts its pipeline for a second phase (measured on the
        // Llama-shaped mixed batch: 91.6 -> 87 us per step), while CTAs without span work keep the
        // CUDA-core body, which is the faster one on decode rows.
        auto line_fill = [&](int path, const std::vector<int>& list, int started) {
            int cta = 0;
            bool has_phase = false;
            // A narrow item costs about 2 us more than an item of the CUDA-core body, a second phase
            // costs about 9 us once: the span CTA keeps to the tensor-core body only if the room left
            // on it takes a few decode units (on the 32-sequence mixed batch, with about two units per
            // span CTA, the step measures 89.3 us with this and 91.8 us without).
            auto rides_along = [&](int k) {
                return k < started && (path == 0 || cap - load[(size_t)k] <= kMaxNarrowUnitsPerCta * avg_unit_ns);
            };
            bool narrow_cta = rides_along(0);
            for (int id : list) {
                const int64_t n_keys = units[id].n_keys;
                int64_t k0 = 0;
                int c = 0;
                while (k0 < n_keys) {
                    const int pth = narrow_cta ? 0 : path;
                    const PathCost& pc = cost[pth];
                    const bool narrow = pth == 0;          // only narrow units are line-filled on the tensor path
                    const int64_t tns = narrow ? narrow_tile_ns : tns_of[(size_t)id];
                    const int64_t item_ns = narrow ? narrow_item_ns : pc.item_ns;
                    const int64_t left = (n_keys - k0 + pc.gran - 1) / pc.gran;
                    const bool last_cta = cta + 1 >= n_ctas;
                    const int64_t start = item_ns + ((has_phase || narrow_cta) ? 0 : pc.phase_ns);
                    const int64_t room = cap - load[(size_t)cta] - start;
                    int64_t take;
                    if (last_cta) {
                        take = left;
                        if (load[(size_t)cta] + start + take * tns > cap) fits = false;
                    } else if (left * tns <= room + item_ns / 2) {
                        take = left;                     // finishing here is cheaper than another item elsewhere
                    } else if (room < tns * 2) {
                        ++cta;                           // not worth starting an item for so little
                        has_phase = false;
                        narrow_cta = rides_along(cta);
                        continue;
                    } else {
                        take = std::max<int64_t>(1, room / tns);
                    }
                    const int64_t k1 = std::min<int64_t>(n_keys, k0 + take * pc.gran);
                    if (emit) out[pth].push_back(Piece{Item{id, (int32_t)k0, (int32_t)k1, c}, (int32_t)cta});
                    else if (!fits) return false;
                    load[(size_t)cta] += start + take * tns;
                    has_phase = true;
                    k0 = k1;
                    ++c;
                    if (!last_cta && k0 < n_keys) { ++cta; has_phase = false; narrow_cta = rides_along(cta); }
                }
            }
            return true;
        };
        // narrow tensor units: on the span CTAs first, then on fresh CTAs (which pay the phase start)
        if (!line_fill(0, tensor_narrow, used)) return false;
        if (!line_fill(1, *ids[1], ids[1]->empty() ? 0 : used)) return false;
        std::stable_sort(out[0].begin(), out[0].end(), [](const Piece& x, const Piece& y) { return x.cta < y.cta; });
        return fits;
    };
    // Smallest limit that fits, by bisection (the loads are monotone in the limit up to rounding).
    // The probes only ask whether a limit fits; the pieces are built once, for the limit found.
    int64_t lo = std::max<int64_t>(1, total / n_ctas * 3 / 4);     // (decode rows on span CTAs cost less than assumed in `total`)
    int64_t hi = lo + lo / 4 + kTensorCost.item_ns + kTensorCost.phase_ns + kCudaCost.phase_ns;
    while (!fill(hi, best, false)) { lo = hi; hi += hi / 2; }
    for (int iter = 0; iter < 24 && hi - lo > std::max<int64_t>(50, hi / 128); ++iter) {      // to 0.8 %
        const int64_t mid = (lo + hi) / 2;
        if (fill(mid, best, false)) hi = mid; else lo = mid;
    }
    fill(hi, best, true);
    // emit: CUDA-core items first, then tensor items; chunk counts per unit
    cta_indptr_cuda.assign((size_t)n_ctas + 1, 0);
    cta_indptr_tensor.assign((size_t)n_ctas + 1, 0);
    for (int path = 1; path >= 0; --path) {
        std::vector<int32_t>& indptr = path == 1 ? cta_indptr_cuda : cta_indptr_tensor;
        const int32_t first = (int32_t)items.size();
        std::vector<int32_t> count((size_t)n_ctas, 0);
        for (const Piece& pz : best[path]) {
            items.push_back(pz.it);
            item_cta.push_back(pz.cta);
            count[(size_t)pz.cta]++;
            units[pz.it.unit].u.n_chunks = std::max(units[pz.it.unit].u.n_chunks, pz.it.chunk + 1);
        }
        int32_t at = first;
        for (int k = 0; k < n_ctas; ++k) {
            indptr[(size_t)k] = at;
            at += count[(size_t)k];
        }
        indptr[(size_t)n_ctas] = at;
    }
}

}  // namespace

extern "C" int asynclm_plan(const asynclm_shape* shape, const asynclm_plan_options* opts,
                            const asynclm_batch* batch, void* host_ws, size_t host_bytes,
                            void* dev_ws, size_t dev_bytes, void* stream,
                            asynclm_plan_t** out_plan) {
    int rc = check_shape(shape);
    if (rc != ASYNCLM_OK) return rc;
    if (!batch || !host_ws || !out_plan || batch->batch < 0) return ASYNCLM_ERR_INVALID_ARG;
    if (((uintptr_t)host_ws & 7) != 0 || ((uintptr_t)dev_ws & 255) != 0)
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
        const int step = tensor ? TQ : 1;
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
    if (fixed_chunk > 0 || ctas_cuda != ctas_tensor) {
        cut_and_deal(ids_cuda, units, fixed_chunk, ctas_cuda, kCudaItemOverheadTiles, items,
                     cta_indptr_cuda, item_cta);
        n_items_cuda = (int)items.size();
        cut_and_deal(ids_tensor, units, fixed_chunk, ctas_tensor, kTensorItemOverheadTiles, items,
                     cta_indptr_tensor, item_cta);
    } else {
        deal_jointly(ids_tensor, ids_cuda, units, G, ctas_cuda, items, cta_indptr_cuda, cta_indptr_tensor, item_cta);
        n_items_cuda = cta_indptr_cuda[(size_t)ctas_cuda];
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

    char* db = (char*)dev_ws;
    DevPlan& d = plan->dev;
    auto dp = [&](size_t off) { return host_only ? nullptr : (void*)(db + off); };
    d.status = (int32_t*)dp(L.off_status);
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
    info.launches_attn = ((n_items_cuda > 0 || d.num_items_tensor > 0) ? 1 : 0) + (d.num_split_units > 0 ? 1 : 0);
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
