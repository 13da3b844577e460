// Host-side ODMA allocator: length buckets, sliding-window quantile boundaries, Large Bucket.
// Plain C++ (no CUDA).  Design section of the paper: III-B (uncertainty), III-C (adaptive
// buckets, Eq. 2), III-D (Large Bucket), III-E (reserve / release), IV-C (integration).
#pragma once

#include <condition_variable>
#include <cstdint>
#include <deque>
#include <map>
#include <memory>
#include <mutex>
#include <thread>
#include <unordered_map>
#include <vector>

#include "odma.h"

namespace odma {

// Free space of one region, kept as address-ordered runs.  Every base and size handed in is a
// multiple of the granule, so every run is too.  take() is lowest-address first fit;
// give() merges with both neighbours at once, so no stale size classes survive a change of
// bucket boundaries.
class FreeRuns {
  public:
    void reset(int64_t lo, int64_t hi);
    int64_t take(int64_t size);          // base of the run taken, or -1
    void give(int64_t base, int64_t size);
    int64_t free_tokens() const { return free_; }
    size_t runs() const { return runs_.size(); }

  private:
    std::map<int64_t, int64_t> runs_;    // base -> length
    int64_t free_ = 0;
};

// Sliding window of the last W realised lengths with an online histogram (a Fenwick tree of
// counts per length) that answers nearest-rank order statistics without sorting.
class LengthWindow {
  public:
    void reset(int32_t window, int32_t max_value);
    void push(int32_t value);
    int32_t count() const { return static_cast<int32_t>(n_); }
    int32_t order_statistic(int64_t rank) const;   // rank in [1, count()]: the rank-th smallest

  private:
    void add(int32_t value, int32_t delta);
    std::vector<int32_t> ring_;
    std::vector<int32_t> tree_;                    // 1-based Fenwick tree over value+1
    int64_t n_ = 0, head_ = 0;
    int32_t top_ = 1;                              // largest power of two <= tree size
};

struct Request {
    int64_t base = 0, cap = 0, len = 0;
    int32_t pool = 0, bucket = 0, migrations = 0;
    uint64_t epoch = 0;
};

struct Migration {        // what the device has to copy after a successful ensure()
    int64_t src_base, src_cap, dst_base, dst_cap, len;
};

class Allocator {
  public:
    Allocator() = default;
    ~Allocator();
    Allocator(const Allocator&) = delete;
    Allocator& operator=(const Allocator&) = delete;
    int32_t init(uint64_t bytes, int32_t layers, int32_t kv_heads, int32_t head_dim,
                 int32_t elem_bytes, const odma_config& cfg);
    int32_t set_buckets(const int32_t* b, int32_t n);
    int32_t get_buckets(int32_t* b, int32_t* n, uint64_t* epoch) const;
    int32_t reserve(uint64_t req, int64_t predicted, odma_slab* out);
    int32_t reserve_uncertain(uint64_t req, int64_t l_hat, int64_t u_pm, odma_slab* out);
    int32_t ensure(uint64_t req, int64_t need, odma_slab* out, int32_t* migrated, Migration* mig);
    int32_t release(uint64_t req);
    int32_t commit(const uint64_t* reqs, int32_t n, const int32_t* n_new);
    const Request* find(uint64_t req) const;
    void stats(odma_stats* out) const;
    // Realised lengths from elsewhere (other replicas, a replayed log) enter the window exactly as
    // local completions do; drain() hands out (and forgets) the lengths completed here since the
    // last drain; flush() returns once the background thread, if any, has applied everything logged.
    int32_t observe(const int32_t* lengths, int32_t n);
    int32_t drain(int32_t* out, int32_t cap, int32_t* n);
    void flush();

    int64_t T() const { return T_; }
    int64_t S() const { return S_; }
    int64_t M() const { return M_; }
    const odma_config& config() const { return cfg_; }
    uint64_t epoch() const;

  private:
    int32_t reserve_large(uint64_t req, int64_t need, odma_slab* out);
    int32_t place_large(int64_t need, int64_t* base, int64_t* cap);
    void recalibrate();
    void apply_observation(int32_t len);     // window + refresh; caller thread (sync) or the background thread
    void note_observation(int32_t len);      // what release() and observe() do with a realised length
    void worker();
    void fill(const Request& r, odma_slab* out) const;
    void note_safety_peak();

    odma_config cfg_{};
    int64_t T_ = 0, S_ = 0, M_ = 0, G_ = 16;
    FreeRuns main_, safety_;
    std::unordered_map<uint64_t, Request> live_;
    LengthWindow window_;
    // boundaries and their epoch: written by recalibrate() (the background thread when async_recal),
    // read by reserve / get_buckets on the caller's thread
    mutable std::mutex bounds_mu_;
    int32_t n_bounds_ = 1;
    int64_t bounds_[ODMA_MAX_BUCKETS] = {0};
    uint64_t epoch_ = 0;
    int64_t applied_ = 0;                    // observations the window has seen (refresh every cfg.refresh of them)
    std::vector<int32_t> outbox_;            // lengths completed here, not yet drained
    // async_recal: release() only logs the length; this thread owns the window
    struct Async {
        std::thread th;
        std::mutex mu;
        std::condition_variable work, idle;
        std::deque<int32_t> log;
        bool stop = false, busy = false;
    };
    std::unique_ptr<Async> async_;
    int64_t observed_ = 0, completed_ = 0, sum_len_ = 0, sum_cap_ = 0, migrations_ = 0, nomem_ = 0,
            routed_large_ = 0, safety_peak_ = 0, reserved_live_ = 0, used_live_ = 0;
};

}  // namespace odma
