// Admission / serving simulator (odma_sim_run): one model replica decoding in lock step over a
// fixed KV pool, requests arriving over time, under one of three reservation policies: static
// worst-case reservation, 16-token pages on demand, or this library's bucket allocator (the
// pool's own Allocator, so boundaries adapt and slabs migrate exactly as in serving).
// The rules are stated at the declaration in odma.h; time is integer nanoseconds throughout.
#include <algorithm>
#include <deque>
#include <vector>

#include "allocator.hpp"
#include "odma.h"

namespace odma {

namespace {

constexpr int64_t kPage = 16;

inline int64_t ceil_page(int64_t x) { return (x + kPage - 1) / kPage * kPage; }

struct Live {
    int32_t req;
    int64_t len, reserved;
};

}  // namespace

int32_t simulate(Allocator& alloc, const odma_sim_params& prm, const odma_sim_request* reqs, int32_t n,
                 odma_sim_result* out) {
    if (!reqs || !out || n < 0 || prm.max_batch < 1 || prm.layers < 1 || prm.base_ns < 0 || prm.ps_per_token < 0)
        return ODMA_ERR_INVALID;
    if (prm.policy < ODMA_SIM_STATIC || prm.policy > ODMA_SIM_ODMA) return ODMA_ERR_INVALID;
    for (int32_t i = 0; i < n; ++i)
        if (reqs[i].prompt < 1 || reqs[i].total <= reqs[i].prompt || reqs[i].predicted < 1 || reqs[i].u_permille > 1000 ||
            (i > 0 && reqs[i].arrival_ns < reqs[i - 1].arrival_ns) || reqs[i].arrival_ns < 0)
            return ODMA_ERR_INVALID;
    const int32_t policy = prm.policy;
    const int64_t pool_tokens = alloc.T(), max_len = alloc.config().max_len;
    odma_sim_result r{};
    std::deque<int32_t> queue;
    for (int32_t i = 0; i < n; ++i) queue.push_back(i);
    std::vector<Live> live;                     // in admission order
    std::vector<size_t> gen;
    int64_t free_tokens = pool_tokens, now = 0;
    bool hold = false;                          // nothing is admitted between a preemption and the next completion

    auto give_back = [&](const Live& l) {
        if (policy == ODMA_SIM_ODMA)
            alloc.release(static_cast<uint64_t>(l.req));
        else
            free_tokens += l.reserved;
    };

    while (!queue.empty() || !live.empty()) {
        // ---- admission: first come first served, no overtaking
        while (!queue.empty() && static_cast<int32_t>(live.size()) < prm.max_batch && !(hold && !live.empty())) {
            const int32_t id = queue.front();
            const odma_sim_request& q = reqs[id];
            if (q.arrival_ns > now) {
                if (!live.empty()) break;
                now = q.arrival_ns;
            }
            bool fits = true, never = false;
            int64_t reserved = 0;
            if (policy == ODMA_SIM_STATIC) {
                if (max_len > pool_tokens || q.total > max_len) never = true;
                else if (free_tokens < max_len) fits = false;
                else reserved = max_len;
            } else if (policy == ODMA_SIM_PAGED16) {
                if (ceil_page(q.total) > pool_tokens) never = true;
                else if (free_tokens < ceil_page(q.prompt)) fits = false;
                else reserved = ceil_page(q.prompt);
            } else {
                odma_slab slab{};
                const int32_t rc = q.u_permille >= 0 ? alloc.reserve_uncertain(static_cast<uint64_t>(id), q.predicted, q.u_permille, &slab)
                                                     : alloc.reserve(static_cast<uint64_t>(id), q.predicted, &slab);
                if (rc == ODMA_ERR_NOMEM) {
                    fits = false;
                } else if (rc != ODMA_OK) {
                    return rc;
                } else {
                    reserved = slab.cap_tok;
                    if (q.prompt > reserved) {                 // predicted below the prompt: grow at once
                        int32_t migrated = 0;
                        Migration mig{};
                        const int32_t rc2 = alloc.ensure(static_cast<uint64_t>(id), q.prompt, &slab, &migrated, &mig);
                        if (rc2 != ODMA_OK) {
                            alloc.release(static_cast<uint64_t>(id));
                            if (live.empty()) never = true; else fits = false;
                        } else {
                            r.migrations += migrated;
                            reserved = slab.cap_tok;
                        }
                    }
                    if (fits && !never) {
                        const uint64_t rid = static_cast<uint64_t>(id);
                        const int32_t grow = q.prompt;
                        alloc.commit(&rid, 1, &grow);
                    }
                }
            }
            if (never) {
                r.failed += 1;
                queue.pop_front();
                continue;
            }
            if (!fits) {
                r.deferred += 1;
                if (live.empty()) {                            // nothing will ever free memory for it
                    r.failed += 1;
                    queue.pop_front();
                    continue;
                }
                break;
            }
            if (policy != ODMA_SIM_ODMA) free_tokens -= reserved;
            queue.pop_front();
            live.push_back({id, q.prompt, reserved});
        }
        if (live.empty()) continue;
        // ---- one decode step: room for every live request's next token
        gen.clear();
        for (size_t k = 0; k < live.size(); ++k) {
            Live& l = live[k];
            if (l.len + 1 > l.reserved) {
                if (policy == ODMA_SIM_PAGED16) {
                    if (free_tokens < kPage) {
                        r.stalls += 1;
                        continue;
                    }
                    free_tokens -= kPage;
                    l.reserved += kPage;
                } else if (policy == ODMA_SIM_ODMA) {
                    odma_slab slab{};
                    int32_t migrated = 0;
                    Migration mig{};
                    const int32_t rc = alloc.ensure(static_cast<uint64_t>(l.req), l.len + 1, &slab, &migrated, &mig);
                    if (rc == ODMA_ERR_NOMEM) {
                        r.stalls += 1;
                        continue;
                    }
                    if (rc != ODMA_OK) return rc;
                    r.migrations += migrated;
                    l.reserved = slab.cap_tok;
                }
            }
            gen.push_back(k);
        }
        if (gen.empty()) {                                     // everybody stalled: the youngest goes back
            const Live l = live.back();
            live.pop_back();
            r.tokens_lost += l.len - reqs[l.req].prompt;
            give_back(l);
            if (live.empty()) {                                // it had the pool to itself and still could not grow
                r.failed += 1;
                hold = false;
                continue;
            }
            hold = true;
            queue.push_front(l.req);
            r.preemptions += 1;
            continue;
        }
        int64_t kv_tokens = 0;
        for (size_t k : gen) kv_tokens += live[k].len + 1;
        const int64_t step_ns = prm.layers * (prm.base_ns + kv_tokens * prm.ps_per_token / 1000);
        now += step_ns;
        for (size_t k : gen) {
            live[k].len += 1;
            if (policy == ODMA_SIM_ODMA) {
                const uint64_t rid = static_cast<uint64_t>(live[k].req);
                const int32_t one = 1;
                alloc.commit(&rid, 1, &one);
            }
        }
        r.steps += 1;
        r.tokens_out += static_cast<int64_t>(gen.size());
        int64_t reserved_now = 0, used_now = 0;
        for (const Live& l : live) {
            reserved_now += l.reserved;
            used_now += l.len;
        }
        r.conc_time += static_cast<int64_t>(live.size()) * step_ns;
        r.reserved_time += reserved_now * step_ns;
        r.used_time += used_now * step_ns;
        // ---- completions
        for (size_t k = 0; k < live.size();) {
            if (live[k].len < reqs[live[k].req].total) {
                ++k;
                continue;
            }
            r.completed += 1;
            r.sum_actual += live[k].len;
            r.sum_reserved += live[k].reserved;
            give_back(live[k]);
            live.erase(live.begin() + static_cast<std::ptrdiff_t>(k));
            hold = false;
        }
    }
    r.makespan_ns = now;
    *out = r;
    return ODMA_OK;
}

}  // namespace odma
