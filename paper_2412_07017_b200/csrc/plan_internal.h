// Host-side plan object and planner constants (internal).
#pragma once
#include <math.h>

#include "asynclm.h"
#include "plan_types.h"

namespace asynclm {

constexpr uint64_t kPlanMagic = 0x4153594e434c4d31ull;   // "ASYNCLM1"

// Persistent CTAs per SM of the CUDA-core attention kernel.
constexpr int kCudaSlotsPerSm = 1;
// Fixed cost of starting an item, in units of one 128-token KV tile, used when balancing CTAs.
constexpr int kCudaItemOverheadTiles = 1;
constexpr int kTensorItemOverheadTiles = 4;   // measured: an item boundary costs the tensor kernel about 4 tiles

// True when the tensor-core attention kernel exists for this head_dim.
bool tensor_path_compiled(int head_dim);

int tensor_tile_tokens(int group);

}  // namespace asynclm

struct asynclm_plan_s {
    uint64_t magic;
    asynclm_shape shape;
    asynclm_plan_info info;
    asynclm::DevPlan dev;
    const asynclm::Unit* h_units;
    const asynclm::Item* h_items;
    const int32_t* h_item_cta;
    const int32_t* h_kv_len_before;
    int32_t h_units_path_split;   // items [0, this) are CUDA-core items, the rest tensor items
    int32_t device;
    int32_t host_only;
    int32_t max_q_len;            // longest span of the step
};
