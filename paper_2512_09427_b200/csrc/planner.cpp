// Split plan for one decode step: deals the batch's KV streams to the persistent CTAs in shares
// of equal cost.
//
// A "stream" is the keys/values of one (request, KV head): one contiguous run in the slab, read
// in 64-token tiles.  Streams longer than a share are cut into pieces that fill one share after
// the other; all others go whole, longest first, to the share with the least load so far.  A
// piece of a cut stream leaves a partial result (running max, sum, unnormalised output) in a
// scratch slot and the CTA that delivers the last piece merges them; a whole stream is written
// out directly.  Costs are in tiles: a tile 1, a stream's start-up 1, a piece of a cut stream 6
// more (see plan_batch).
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

    // Shares.  The streams are dealt into at most `ctas` shares of (nearly) equal COST:
    //   * a tile of 64 tokens costs 1;
    //   * starting a stream (its query, its first rows in a new part of memory, handing its
    //     result over) costs kStreamCostTiles;
    //   * a piece of a split stream costs kSplitCostTiles on top: its partial result goes
    //     through global memory and the CTA that delivers the last piece merges them all, a
    //     chain of dependent round trips that a CTA ending on such a piece cannot hide.
    // With capacity C = the average cost per share: "long" streams fill one share after the
    // other, whole where they fit, cut where they do not (no piece shorter than
    // kMinPieceTiles); every other stream goes whole, longest first, to the share with the
    // least load so far (small streams level the shares out).  Long means longer than a share;
    // if that leaves shares overfilled (many streams of between half a share and a share, which
    // do not pack), the plan is redone with long = longer than half a share.
    std::vector<int32_t> order(static_cast<size_t>(n));
    for (int32_t i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return in.len[x] > in.len[y]; });

    struct Piece { int32_t w[8]; int32_t share; };
    std::vector<Piece> pieces;
    std::vector<int32_t> comb;      // {req, head, first_slot, n_slots}
    std::vector<int64_t> load;
    // deal(C, false) cuts the long streams only and returns the number of pieces (-1: more
    // than `ctas` shares needed); deal(C, true) emits the whole plan.
    auto deal = [&](int64_t C, bool emit, int64_t long_div) -> int64_t {
        int64_t n_cut = 0;
        load.assign(static_cast<size_t>(ctas), 0);
        int32_t fresh = 0;          // the share that pieces of long streams are filling
        if (emit) {
            pieces.clear();
            comb.clear();
        }
        auto put = [&](int32_t r, int32_t head, int64_t tile0, int64_t ntiles, bool whole, int32_t share) {
            if (!emit) return;
            const int64_t tok0 = tile0 * kTileTokens;
            const int64_t tok1 = std::min<int64_t>((tile0 + ntiles) * kTileTokens, in.len[r]);
            Piece pc;
            pc.w[0] = r;
            pc.w[1] = head;
            pc.w[2] = static_cast<int32_t>(tok0);
            pc.w[3] = static_cast<int32_t>(tok1 - tok0);
            pc.w[4] = (whole ? 1 : 0) | (tok1 == in.len[r] ? 2 : 0);   // bit 0 direct, bit 1 ends its stream
            pc.w[5] = static_cast<int32_t>(pieces.size());       // slot
            // first row of the piece inside one K (or V) array of the pool
            pc.w[6] = static_cast<int32_t>(static_cast<int64_t>(in.base[r]) * hkv +
                                           static_cast<int64_t>(head) * in.cap[r] + tok0);
            pc.w[7] = -1;                                          // combine record, set below
            pc.share = share;
            pieces.push_back(pc);
        };
        auto record_split = [&](int32_t r, int32_t head, int32_t first_slot) {
            const int32_t n_pieces = static_cast<int32_t>(pieces.size()) - first_slot;
            const int32_t ci = static_cast<int32_t>(comb.size() / 4);
            for (int32_t j = first_slot; j < first_slot + n_pieces; ++j) pieces[j].w[7] = ci;
            comb.push_back(r);
            comb.push_back(head);
            comb.push_back(first_slot);
            comb.push_back(n_pieces);
        };
        // long streams first (the order is by length), filling one share after the other; a
        // stream's last piece leaves room that the next stream, or short streams later, take
        int32_t oi = 0;
        for (; oi < n; ++oi) {
            const int32_t r = order[oi];
            const int64_t per = (in.len[r] + kTileTokens - 1) / kTileTokens;
            if (long_div * (per + kStreamCostTiles) <= C || per < 2 * kMinPieceTiles) break;
            for (int32_t head = 0; head < hkv; ++head) {
                if (fresh < ctas && load[fresh] + per + kStreamCostTiles <= C) {     // fits whole
                    put(r, head, 0, per, true, fresh);
                    load[fresh] += per + kStreamCostTiles;
                    continue;
                }
                const int32_t first_slot = static_cast<int32_t>(pieces.size());
                int64_t done = 0;
                while (done < per) {
                    if (fresh >= ctas) return -1;
                    const int64_t extra = kSplitCostTiles + (done == 0 ? kStreamCostTiles : 0);
                    int64_t room = C - load[fresh] - extra;
                    if (room < kMinPieceTiles && load[fresh] > 0) {          // this share is full
                        ++fresh;
                        continue;
                    }
                    int64_t take = std::min(std::max<int64_t>(room, 1), per - done);
                    if (per - done - take > 0 && per - done - take < kMinPieceTiles)
                        take = std::max<int64_t>(1, per - done - kMinPieceTiles);   // no crumbs
                    put(r, head, done, take, false, fresh);
                    ++n_cut;
                    load[fresh] += take + extra;
                    done += take;
                    if (done < per) ++fresh;
                }
                if (emit) {
                    if (static_cast<int32_t>(pieces.size()) - first_slot > 1)
                        record_split(r, head, first_slot);
                    else
                        pieces[first_slot].w[4] |= 1;      // moved to a fresh share and fitted whole
                }
            }
        }
        if (!emit) return n_cut;
        // every other stream whole, longest first, to the least loaded share: shares are kept
        // in buckets by load (loads are small integers), the least loaded bucket is found by
        // a pointer that only moves up
        int64_t top = 0;
        for (int32_t c = 0; c < ctas; ++c) top = std::max(top, load[c]);
        std::vector<std::vector<int32_t>> bucket(static_cast<size_t>(top) + 2);
        for (int32_t c = ctas - 1; c >= 0; --c) bucket[static_cast<size_t>(load[c])].push_back(c);
        size_t lo = 0;
        auto least = [&]() {
            while (bucket[lo].empty()) ++lo;
            const int32_t c = bucket[lo].back();
            bucket[lo].pop_back();
            return c;
        };
        auto back = [&](int32_t c) {
            if (static_cast<size_t>(load[c]) >= bucket.size()) bucket.resize(static_cast<size_t>(load[c]) + 1);
            bucket[static_cast<size_t>(load[c])].push_back(c);
        };
        for (; oi < n; ++oi) {
            const int32_t r = order[oi];
            const int64_t per = (in.len[r] + kTileTokens - 1) / kTileTokens;
            for (int32_t head = 0; head < hkv; ++head) {
                int32_t c = least();
                if (load[c] == 0 || load[c] + per + kStreamCostTiles <= C + kSlackTiles || per < 2 * kMinPieceTiles) {
                    put(r, head, 0, per, true, c);
                    load[c] += per + kStreamCostTiles;
                    back(c);
                    continue;
                }
                // it would overfill even the least loaded share: cut it over the least loaded ones
                const int32_t first_slot = static_cast<int32_t>(pieces.size());
                int64_t done = 0;
                while (done < per) {
                    const int64_t extra = kSplitCostTiles + (done == 0 ? kStreamCostTiles : 0);
                    const int64_t room = C - load[c] - extra;
                    int64_t take = per - done;
                    if (room >= std::max<int64_t>(kMinPieceTiles, per / 2) && room < take) {   // two pieces at most
                        take = room;
                        if (per - done - take < kMinPieceTiles) take = std::max<int64_t>(1, per - done - kMinPieceTiles);
                    }
                    put(r, head, done, take, false, c);
                    load[c] += take + extra;
                    back(c);
                    done += take;
                    if (done < per) c = least();
                }
                if (static_cast<int32_t>(pieces.size()) - first_slot > 1)
                    record_split(r, head, first_slot);
                else
                    pieces[first_slot].w[4] |= 1;      // no share had room for a piece: whole after all
            }
        }
        return n_cut;
    };
    int64_t cost = 0;
    for (int32_t i = 0; i < n; ++i)
        cost += ((in.len[i] + kTileTokens - 1) / kTileTokens + kStreamCostTiles) * hkv;
    // the capacity is the average cost per share, split costs included (a few rounds: the
    // number of pieces depends on the capacity)
    for (int64_t long_div = 1; long_div <= 2; ++long_div) {
        // the capacity is the average cost per share, split costs included (a few rounds: the
        // number of pieces depends on the capacity)
        int64_t C = std::max<int64_t>((cost + ctas - 1) / ctas, 1 + kStreamCostTiles);
        for (int round = 0; round < 64; ++round) {
            const int64_t n_cut = deal(C, false, long_div);
            const int64_t want = n_cut < 0 ? C + C / 128 + 1 : (cost + n_cut * kSplitCostTiles + ctas - 1) / ctas;
            if (n_cut >= 0 && want <= C) break;
            C = std::max(want, C + 1);
        }
        if (deal(C, true, long_div) < 0) return ODMA_ERR_INVALID;
        int64_t worst = 0;
        for (int32_t c = 0; c < ctas; ++c) worst = std::max(worst, load[c]);
        if (worst <= C + kSlackTiles + C / 16) break;
    }
    const int32_t n_items = static_cast<int32_t>(pieces.size());
    // the table was sized for at most streams + ctas items and min(streams, ctas) cut streams
    if (static_cast<int64_t>(t.off_items) + 8ll * n_items + static_cast<int64_t>(comb.size()) > table_words)
        return ODMA_ERR_INVALID;

    // Group the pieces by share.  Each CTA works through its pieces of split streams first,
    // then through the whole streams: partial results are delivered early, so the merge of a
    // split stream overlaps with streaming instead of trailing the kernel.
    std::vector<int32_t> count(static_cast<size_t>(ctas) + 1, 0);
    for (const Piece& pc : pieces) ++count[pc.share + 1];
    int32_t used = 0;
    for (int32_t c = 0; c < ctas; ++c)
        if (count[c + 1] > 0) used = c + 1;
    std::vector<int32_t> at(static_cast<size_t>(ctas) + 1, 0);
    for (int32_t c = 0; c < ctas; ++c) at[c + 1] = at[c] + count[c + 1];
    std::vector<int32_t> fill(at.begin(), at.end() - 1);
    for (int pass = 0; pass < 2; ++pass)
        for (const Piece& pc : pieces)
            if (((pc.w[4] & 1) == 0) == (pass == 0)) {
                std::copy(pc.w, pc.w + 8, items + 8 * fill[pc.share]);
                ++fill[pc.share];
            }
    for (int32_t c = 0; c < used; ++c) {
        int32_t* rec = table + t.off_cta + kCtaWords * c;
        rec[0] = at[c];
        rec[1] = at[c + 1];
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
    t.n_ctas = used;
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
