// Split plan for one decode step: cuts the batch's KV streams into equal shares of tiles.
//
// A "stream" is the keys/values of one (request, KV head): one contiguous run in the slab.
// All streams of the batch, laid end to end in (request, head) order, form a sequence of
// 64-token tiles.  The plan gives each persistent CTA a contiguous share of that sequence, so
// every CTA streams the same number of bytes (+-1 tile) whatever the length mix of the batch.
// A share that ends inside a stream leaves a partial result (running max, sum, unnormalised
// output) in a scratch slot; a stream covered by one share is written out directly.
#include "planner.hpp"

#include <algorithm>

namespace odma {

static inline int32_t align4(int32_t w) { return (w + 3) & ~3; }

int64_t plan_table_words(int32_t n, int32_t kv_heads, int32_t n_ctas) {
    const int64_t streams = static_cast<int64_t>(n) * kv_heads;
    int64_t w = 0;
    w += align4(n) * 3;                 // base, cap, len
    w += align4(n + 1);                 // cu_new
    w += kCtaWords * n_ctas;            // per-CTA records
    w += 8 * (streams + n_ctas);        // items
    w += 4 * std::min<int64_t>(streams, n_ctas);   // combine records
    return w;
}

int32_t plan_batch(const PlanInput& in, int32_t* table, int64_t table_words, odma_tables* out) {
    const int32_t n = in.n, hkv = in.kv_heads;
    if (n < 1 || hkv < 1 || in.n_ctas < 1) return ODMA_ERR_INVALID;
    if (plan_table_words(n, hkv, in.n_ctas) > table_words) return ODMA_ERR_INVALID;

    // tiles per stream and in total
    std::vector<int64_t> first_tile(static_cast<size_t>(n) + 1, 0);   // per request, all heads
    int64_t kv_tokens = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (in.len[i] < 1) return ODMA_ERR_INVALID;
        const int64_t tiles = (in.len[i] + kTileTokens - 1) / kTileTokens;
        first_tile[i + 1] = first_tile[i] + tiles * hkv;
        kv_tokens += in.len[i];
    }
    const int64_t total = first_tile[n];
    const int32_t ctas = static_cast<int32_t>(std::min<int64_t>(in.n_ctas, total));

    // word layout
    odma_tables t{};
    int32_t w = 0;
    t.off_base = w;       w += align4(n);
    t.off_cap = w;        w += align4(n);
    t.off_len = w;        w += align4(n);
    t.off_cu_new = w;     w += align4(n + 1);
    t.off_cta = w;        w += kCtaWords * ctas;
    t.off_items = w;
    int32_t* items = table + t.off_items;

    int32_t cu = 0;
    bool one_each = true;
    for (int32_t i = 0; i < n; ++i) {
        one_each = one_each && (!in.n_new || in.n_new[i] == 1);
        table[t.off_base + i] = in.base[i];
        table[t.off_cap + i] = in.cap[i];
        table[t.off_len + i] = in.len[i];
        table[t.off_cu_new + i] = cu;
        cu += in.n_new ? in.n_new[i] : 1;
    }
    table[t.off_cu_new + n] = cu;

    // Cut points.  Shares are equal in COST, not in tiles: starting a stream (its query, its
    // first rows in a new part of memory, its merge at the end) costs about as much as
    // streaming kStreamCostTiles more tiles, so a stream of `per` tiles weighs per +
    // kStreamCostTiles.  A cut that falls into a stream's start-up part moves to the stream's
    // start, one that falls inside a short stream moves to its nearer end.
    std::vector<int64_t> first_cost(static_cast<size_t>(n) + 1, 0);
    for (int32_t i = 0; i < n; ++i)
        first_cost[i + 1] = first_cost[i] + ((first_tile[i + 1] - first_tile[i]) / hkv + kStreamCostTiles) * hkv;
    const int64_t total_cost = first_cost[n];
    std::vector<int64_t> cut(static_cast<size_t>(ctas) + 1);
    cut[0] = 0;
    cut[ctas] = total;
    int32_t req = 0;
    for (int32_t c = 1; c < ctas; ++c) {
        const int64_t xc = total_cost * c / ctas;
        while (first_cost[req + 1] <= xc) ++req;                    // request holding cost unit xc
        const int64_t per = (first_tile[req + 1] - first_tile[req]) / hkv;   // tiles per stream
        const int64_t per_cost = per + kStreamCostTiles;
        const int64_t sh = (xc - first_cost[req]) / per_cost;       // stream of that request
        const int64_t off = (xc - first_cost[req]) - sh * per_cost - kStreamCostTiles;
        const int64_t s0 = first_tile[req] + sh * per, s1 = s0 + per;
        int64_t x = s0 + std::max<int64_t>(off, 0);
        if (per <= kSnapTiles) x = (x - s0 <= s1 - x) ? s0 : s1;
        cut[c] = std::max(x, cut[c - 1]);
    }

    // walk the tile sequence once, emitting one piece per (share, stream) overlap, in stream
    // order; a piece's slot (where its partial result goes) is its index in that order
    struct Piece { int32_t w[8]; };
    std::vector<Piece> pieces;
    std::vector<int32_t> share_begin(static_cast<size_t>(ctas) + 1, 0);
    std::vector<int32_t> comb;      // {req, head, first_slot, n_slots}
    int32_t r = 0, head = 0;
    int64_t stream_lo = 0;          // first tile of the current stream
    int64_t pos = 0;
    int32_t stream_first = 0;
    for (int32_t c = 0; c < ctas; ++c) {
        share_begin[c] = static_cast<int32_t>(pieces.size());
        while (pos < cut[c + 1]) {
            const int64_t per = (in.len[r] + kTileTokens - 1) / kTileTokens;
            const int64_t stream_hi = stream_lo + per;
            const int64_t end = std::min(stream_hi, cut[c + 1]);
            const int64_t tok0 = (pos - stream_lo) * kTileTokens;
            const int64_t tok1 = std::min<int64_t>((end - stream_lo) * kTileTokens, in.len[r]);
            const int32_t k = static_cast<int32_t>(pieces.size());
            Piece pc;
            pc.w[0] = r;
            pc.w[1] = head;
            pc.w[2] = static_cast<int32_t>(tok0);
            pc.w[3] = static_cast<int32_t>(tok1 - tok0);
            pc.w[4] = (pos == stream_lo && end == stream_hi) ? 1 : 0;    // whole stream: direct
            pc.w[5] = k;                                                 // slot
            // first row of the piece inside one K (or V) array of the pool
            pc.w[6] = static_cast<int32_t>(static_cast<int64_t>(in.base[r]) * hkv +
                                           static_cast<int64_t>(head) * in.cap[r] + tok0);
            pc.w[7] = -1;                                                // combine record, set below
            if (pos == stream_lo) stream_first = k;
            pieces.push_back(pc);
            pos = end;
            if (end == stream_hi) {                                      // stream finished
                const int32_t n_pieces = static_cast<int32_t>(pieces.size()) - stream_first;
                if (n_pieces > 1) {
                    const int32_t ci = static_cast<int32_t>(comb.size() / 4);
                    for (int32_t j = stream_first; j < stream_first + n_pieces; ++j) pieces[j].w[7] = ci;
                    comb.push_back(r);
                    comb.push_back(head);
                    comb.push_back(stream_first);
                    comb.push_back(n_pieces);
                }
                stream_lo = stream_hi;
                if (++head == hkv) {
                    head = 0;
                    ++r;
                }
            }
        }
    }
    share_begin[ctas] = static_cast<int32_t>(pieces.size());
    const int32_t n_items = static_cast<int32_t>(pieces.size());

    // Each CTA works through the pieces of split streams first (at most its first and its last
    // piece), then through the whole streams: partial results are delivered early, so the
    // merge of a split stream overlaps with streaming instead of trailing the kernel.
    int32_t out_i = 0;
    for (int32_t c = 0; c < ctas; ++c) {
        int32_t* rec = table + t.off_cta + kCtaWords * c;
        rec[0] = out_i;
        for (int pass = 0; pass < 2; ++pass)
            for (int32_t k = share_begin[c]; k < share_begin[c + 1]; ++k)
                if ((pieces[k].w[4] == 0) == (pass == 0)) {
                    std::copy(pieces[k].w, pieces[k].w + 8, items + 8 * out_i);
                    ++out_i;
                }
        rec[1] = out_i;
        rec[2] = rec[3] = 0;
        // a copy of the CTA's first item rides in its record: one load starts its stream
        for (int k = 0; k < 8; ++k) rec[4 + k] = rec[0] < rec[1] ? items[8 * rec[0] + k] : 0;
    }
    w = t.off_items + 8 * n_items;
    t.off_combine = w;
    std::copy(comb.begin(), comb.end(), table + w);
    w += static_cast<int32_t>(comb.size());

    t.d_table = nullptr;
    t.n = n;
    t.n_new_total = cu;
    t.n_items = n_items;
    t.n_ctas = ctas;
    t.n_combine = static_cast<int32_t>(comb.size() / 4);
    t.words = w;
    t.tile_tokens = kTileTokens;
    t.one_new_each = one_each ? 1 : 0;
    t.kv_tokens = kv_tokens;
    t.epoch = 0;
    *out = t;
    return ODMA_OK;
}

}  // namespace odma
