// Internal plan format shared by the host planner and the kernels (not part of the public ABI).
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace asynclm {

constexpr int kKvTile = 128;          // split-KV chunk granularity in tokens (8 pages of 16)
constexpr int kPage = 16;
constexpr int kPathCuda = 0;         // the warp-level body (decode rows, short spans)
constexpr int kPathTensor = 1;

// A unit is one query tile of one (sequence, kv head): `ntok` consecutive new tokens times the G
// query heads that share the kv head.  Token t of the unit sees keys [0, kv_limit0 + t).
struct Unit {
    int32_t seq;
    int32_t kv_head;
    int32_t q_row0;        // global token row of the unit's first token
    int32_t ntok;
    int32_t kv_limit0;     // ctx_b + tok0 + 1
    int32_t n_chunks;      // number of KV chunks (items) of this unit
    int32_t partial_base;  // first partial row (chunk c, token t -> partial_base + c*ntok + t); -1 if unsplit
    int32_t page_base;     // page_indptr[seq]
};

// An item is one KV chunk of one unit.
struct Item {
    int32_t unit;
    int32_t kv0;           // first key position
    int32_t kv1;           // one past the last key position any token of the unit may see here
    int32_t chunk;         // chunk index inside the unit
};

// What an attention kernel needs to run one item, resolved by the planner so that a CTA reaches its
// first page ids with two dependent loads (its item range, then this record).
struct alignas(16) Work {
    int32_t kv0;           // first key position
    int32_t kv_end;        // one past the last key any token of the unit sees in this item
    int32_t q_row0;        // global token row of the unit's first token
    int32_t ntok;
    int32_t kv_limit0;     // token t of the unit sees keys [0, kv_limit0 + t)
    int32_t kv_head;
    int32_t partial_row0;  // partial row of token 0 in this chunk; -1: the item writes final output
    int32_t page0;         // index into page_indices of the page that holds key kv0
    int32_t unit;          // the unit this item is a chunk of
    int32_t n_chunks;      // chunks of that unit
    int32_t partial_base;  // partial row of its chunk 0, token 0 (-1 if unsplit)
    int32_t q_seq0;        // global token row of the sequence's first new token (its position is
                           // ctx = kv_limit0 - 1 - (q_row0 - q_seq0))
};

// Per persistent CTA, one 384-byte header that holds everything the CTA needs to issue its first
// loads after a single round trip to memory: words 0-3 its item ranges (span body first, last;
// warp body first, last), words 8-19 the Work record of its first span item, words 20-31 that of
// its first warp-body item, words 32-63 the first 32 page ids of the first span item and words
// 64-95 those of the first warp-body item.
constexpr int kHeadWords = 96;
constexpr int kHeadWorkTensor = 8, kHeadWorkCuda = 20, kHeadPagesTensor = 32, kHeadPagesCuda = 64;

// The new K/V rows of the step, for attention kernels that append them themselves (asynclm_step);
// k_new == nullptr: the rows are in the pool already.
struct AppendSrc {
    const void* k_new;     // bf16 [T][Hkv][d]
    const void* v_new;
    void* pool;            // the pool, writable
};

// Pointers into the device workspace, passed to kernels by value.
struct DevPlan {
    const int32_t* q_indptr;
    const int32_t* kv_len_before;
    const int32_t* page_indptr;
    const int32_t* page_indices;
    const int32_t* row_seq;          // [T] sequence of each new token row
    const int64_t* row_slot;         // [T] page * 16 + slot where the row's K/V go (resolved by the planner)
    const Unit* units;
    const Item* items;               // CUDA-core items first (grouped by CTA), then tensor items
    const Work* works;               // [num_items] the same items, resolved for the kernels
    const int32_t* cta_heads;        // [num_ctas][kHeadWords], see above
    const int32_t* cta_indptr_cuda;  // [num_ctas_cuda + 1] into items
    const int32_t* cta_indptr_tensor;// [num_ctas_tensor + 1] into items (absolute indices)
    const int32_t* split_units;      // [num_split_units] unit ids whose keys were cut into chunks
    const int32_t* merge_blocks;     // [num_merge_blocks] (unit id << 6) | row block: 4 (token, head) rows each,
                                     // for the split units of the span body (the merge kernel's work list)
    int32_t* unit_arrivals;          // [num_units] chunks of a split warp-body unit that have written their
                                     // partial rows; the CTA that brings a count to n_chunks merges the unit
                                     // and puts the count back to zero
    float* partial_o;                // [partial_rows][G][d]
    float* partial_lse;              // [partial_rows][G]   (log2 domain)
    int32_t* status;                 // device status word
    int32_t* counters;               // [0] next chunk of the warp body's queue, [1] CTAs that are done with the
                                     // queue; both are zero between launches (the last CTA puts them back)
    int32_t queue_first, queue_count;// items [queue_first, queue_first + queue_count) are handed out at run time
    int32_t batch, total_q, num_units, num_items, num_items_cuda, num_items_tensor;
    int32_t num_split_units, num_ctas_cuda, num_ctas_tensor;
    int32_t num_merge_blocks;
    int32_t num_q_heads, num_kv_heads, head_dim, group;
    int64_t num_pages;
    float sm_scale;
    int32_t debug_stall_tile;        // checked build only, 0 = off: the K producer of CTA 0 leaves out the hand-off
                                     // of its n-th span tile, so that the wait for it runs out (see api.cu)
};

}  // namespace asynclm
