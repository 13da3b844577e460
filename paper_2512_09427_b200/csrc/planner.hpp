// Split plan for one decode step (see planner.cpp).
#pragma once

#include <cstdint>
#include <vector>

#include "odma.h"

namespace odma {

constexpr int32_t kTileTokens = 64;   // tokens staged per pipeline stage
constexpr int32_t kSnapTiles = 2;     // streams this short are never cut in two
constexpr int32_t kStreamCostTiles = 1;  // a stream's start-up weighs as much as this many tiles
constexpr int32_t kSplitCostTiles = 6;   // so does, on top, every piece of a split stream
constexpr int32_t kMinPieceTiles = 3;    // no piece of a split stream is shorter than this
constexpr int32_t kSlackTiles = 2;       // a whole stream may overfill a share by this much rather than be cut
constexpr int32_t kCtaWords = 12;     // per-CTA record: {item_begin, item_end, 0, 0, first item[8]}

struct PlanInput {
    int32_t n = 0, kv_heads = 0, n_ctas = 0;
    const int32_t* base = nullptr;    // per request: slab base, capacity, length after the append
    const int32_t* cap = nullptr;
    const int32_t* len = nullptr;
    const int32_t* n_new = nullptr;   // tokens appended this step (nullptr = 1 each)
};

// Upper bound, in int32 words, of the table plan_batch writes for n requests.
int64_t plan_table_words(int32_t n, int32_t kv_heads, int32_t n_ctas);

// Fills `table` (host memory) and the descriptor; d_table and epoch are left for the caller.
int32_t plan_batch(const PlanInput& in, int32_t* table, int64_t table_words, odma_tables* out);

}  // namespace odma
