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

    // cut points: equal shares, moved to a stream boundary when they fall inside a short stream
    std::vector<int64_t> cut(static_cast<size_t>(ctas) + 1);
    cut[0] = 0;
    cut[ctas] = total;
    int32_t req = 0;
    for (int32_t c = 1; c < ctas; ++c) {
        int64_t x = total * c / ctas;
        while (first_tile[req + 1] <= x) ++req;                     // request holding tile x
        const int64_t per = (first_tile[req + 1] - first_tile[req]) / hkv;   // tiles per stream
        const int64_t s0 = first_tile[req] + (x - first_tile[req]) / per * per;
        const int64_t s1 = s0 + per;
        if (per <= kSnapTiles) x = (x - s0 <= s1 - x) ? s0 : s1;
        cut[c] = std::max(x, cut[c - 1]);
    }

    // walk the tile sequence once, emitting one item per (share, stream) overlap
    int32_t n_items = 0;
    std::vector<int32_t> comb;      // {req, head, first_slot, n_slots}
    int32_t r = 0, head = 0;
    int64_t stream_lo = 0;          // first tile of the current stream
    int64_t pos = 0;
    int32_t stream_first_item = 0;
    for (int32_t c = 0; c < ctas; ++c) {
        int32_t* rec = table + t.off_cta + kCtaWords * c;
        rec[0] = n_items;
        while (pos < cut[c + 1]) {
            const int64_t per = (in.len[r] + kTileTokens - 1) / kTileTokens;
            const int64_t stream_hi = stream_lo + per;
            const int64_t end = std::min(stream_hi, cut[c + 1]);
            const int64_t tok0 = (pos - stream_lo) * kTileTokens;
            const int64_t tok1 = std::min<int64_t>((end - stream_lo) * kTileTokens, in.len[r]);
            int32_t* it = items + 8 * n_items;
            it[0] = r;
            it[1] = head;
            it[2] = static_cast<int32_t>(tok0);
            it[3] = static_cast<int32_t>(tok1 - tok0);
            it[4] = (pos == stream_lo && end == stream_hi) ? 1 : 0;    // whole stream: direct
            it[5] = n_items;                                           // slot = item index
            // first row of the piece inside one K (or V) array of the pool
            it[6] = static_cast<int32_t>(static_cast<int64_t>(in.base[r]) * hkv +
                                         static_cast<int64_t>(head) * in.cap[r] + tok0);
            it[7] = -1;                                                // combine record, set below
            if (pos == stream_lo) stream_first_item = n_items;
            ++n_items;
            pos = end;
            if (end == stream_hi) {                                    // stream finished
                const int32_t pieces = n_items - stream_first_item;
                if (pieces > 1) {
                    const int32_t ci = static_cast<int32_t>(comb.size() / 4);
                    for (int32_t k = stream_first_item; k < n_items; ++k) items[8 * k + 7] = ci;
                    comb.push_back(r);
                    comb.push_back(head);
                    comb.push_back(stream_first_item);
                    comb.push_back(pieces);
                }
                stream_lo = stream_hi;
                if (++head == hkv) {
                    head = 0;
                    ++r;
                }
            }
        }
        rec[1] = n_items;
        rec[2] = rec[3] = 0;
    }
    // a copy of each CTA's first item rides in its record: one load starts the CTA's stream
    for (int32_t c = 0; c < ctas; ++c) {
        int32_t* rec = table + t.off_cta + kCtaWords * c;
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
