// Host-side ODMA allocator (see allocator.hpp).
#include "allocator.hpp"

#include <algorithm>

namespace odma {

static inline int64_t ceil_g(int64_t x, int64_t g) { return (x + g - 1) / g * g; }
static inline int64_t floor_g(int64_t x, int64_t g) { return x / g * g; }

// ---------------------------------------------------------------------------------------------
// FreeRuns
// ---------------------------------------------------------------------------------------------

void FreeRuns::reset(int64_t lo, int64_t hi) {
    runs_.clear();
    free_ = 0;
    if (hi > lo) {
        runs_[lo] = hi - lo;
        free_ = hi - lo;
    }
}

int64_t FreeRuns::take(int64_t size) {
    for (auto it = runs_.begin(); it != runs_.end(); ++it) {
        if (it->second >= size) {
            int64_t base = it->first, rest = it->second - size;
            runs_.erase(it);
            if (rest > 0) runs_[base + size] = rest;
            free_ -= size;
            return base;
        }
    }
    return -1;
}

void FreeRuns::give(int64_t base, int64_t size) {
    free_ += size;
    auto next = runs_.lower_bound(base);
    if (next != runs_.begin()) {
        auto prev = std::prev(next);
        if (prev->first + prev->second == base) {   // merge with the run below
            base = prev->first;
            size += prev->second;
            runs_.erase(prev);
        }
    }
    if (next != runs_.end() && base + size == next->first) {   // and with the run above
        size += next->second;
        runs_.erase(next);
    }
    runs_[base] = size;
}

// ---------------------------------------------------------------------------------------------
// LengthWindow
// ---------------------------------------------------------------------------------------------

void LengthWindow::reset(int32_t window, int32_t max_value) {
    ring_.assign(static_cast<size_t>(window), 0);
    tree_.assign(static_cast<size_t>(max_value) + 2, 0);
    n_ = 0;
    head_ = 0;
    top_ = 1;
    while (static_cast<size_t>(top_) * 2 < tree_.size()) top_ *= 2;
}

void LengthWindow::add(int32_t value, int32_t delta) {
    for (size_t i = static_cast<size_t>(value) + 1; i < tree_.size(); i += i & (~i + 1))
        tree_[i] += delta;
}

void LengthWindow::push(int32_t value) {
    const int64_t w = static_cast<int64_t>(ring_.size());
    if (n_ == w) {                       // the oldest value leaves
        add(ring_[static_cast<size_t>(head_)], -1);
        n_ -= 1;
    }
    ring_[static_cast<size_t>(head_)] = value;
    head_ = (head_ + 1) % w;
    add(value, +1);
    n_ += 1;
}

int32_t LengthWindow::order_statistic(int64_t rank) const {
    // smallest value v with (number of entries <= v) >= rank: descend the Fenwick tree
    size_t pos = 0;
    int64_t left = rank;
    for (size_t step = static_cast<size_t>(top_); step > 0; step >>= 1) {
        size_t nxt = pos + step;
        if (nxt < tree_.size() && tree_[nxt] < left) {
            pos = nxt;
            left -= tree_[nxt];
        }
    }
    return static_cast<int32_t>(pos);    // tree index pos+1 holds value pos
}

// ---------------------------------------------------------------------------------------------
// Allocator
// ---------------------------------------------------------------------------------------------

int32_t Allocator::init(uint64_t bytes, int32_t layers, int32_t kv_heads, int32_t head_dim,
                        int32_t elem_bytes, const odma_config& cfg) {
    if (layers < 1 || kv_heads < 1 || head_dim < 1 || elem_bytes < 1) return ODMA_ERR_INVALID;
    if (cfg.granule < 16 || cfg.granule % 16 != 0) return ODMA_ERR_INVALID;
    if (cfg.max_len < cfg.granule || cfg.max_len % cfg.granule != 0) return ODMA_ERR_INVALID;
    if (cfg.n_levels < 1 || cfg.n_levels > ODMA_MAX_BUCKETS) return ODMA_ERR_INVALID;
    if (cfg.window < 1 || cfg.refresh < 1 || cfg.p_den < 1) return ODMA_ERR_INVALID;
    if (cfg.safety_pct < 0 || cfg.safety_pct > 100 || cfg.growth < 1) return ODMA_ERR_INVALID;
    for (int i = 0; i < cfg.n_levels; ++i)
        if (cfg.p_num[i] < 0) return ODMA_ERR_INVALID;
    cfg_ = cfg;
    G_ = cfg.granule;
    const uint64_t per_tok = static_cast<uint64_t>(layers) * 2u * static_cast<uint64_t>(kv_heads) *
                             static_cast<uint64_t>(head_dim) * static_cast<uint64_t>(elem_bytes);
    T_ = floor_g(static_cast<int64_t>(bytes / per_tok), G_);
    S_ = floor_g(T_ * cfg.safety_pct / 100, G_);
    M_ = T_ - S_;
    if (T_ >= (int64_t(1) << 31)) return ODMA_ERR_INVALID;
    main_.reset(0, M_);
    safety_.reset(M_, T_);
    window_.reset(cfg.window, cfg.max_len);
    live_.clear();
    n_bounds_ = 1;
    bounds_[0] = cfg.max_len;
    epoch_ = 0;
    applied_ = 0;
    outbox_.clear();
    if (cfg.async_recal < 0 || cfg.async_recal > 1 || cfg.cluster_observe < 0 || cfg.cluster_observe > 1)
        return ODMA_ERR_INVALID;
    if (cfg.readout < ODMA_READOUT_AUTO || cfg.readout > ODMA_READOUT_AT_ONCE) return ODMA_ERR_INVALID;
    if (cfg.async_recal) {
        async_.reset(new Async());
        async_->th = std::thread([this] { worker(); });
    }
    observed_ = completed_ = sum_len_ = sum_cap_ = migrations_ = nomem_ = routed_large_ = 0;
    safety_peak_ = reserved_live_ = used_live_ = 0;
    return ODMA_OK;
}

Allocator::~Allocator() {
    if (async_) {
        {
            std::lock_guard<std::mutex> g(async_->mu);
            async_->stop = true;
        }
        async_->work.notify_all();
        if (async_->th.joinable()) async_->th.join();
    }
}

// Background refresh (Sections III-E and IV-C: histogram updates and boundary refreshes run off
// the critical path; new boundaries reach newly admitted requests only, which holds by
// construction: a slab is sized once, at admission).  The thread applies the logged lengths in
// order, so at quiescence the boundaries are those the synchronous path would have.
void Allocator::worker() {
    Async& a = *async_;
    std::unique_lock<std::mutex> lk(a.mu);
    for (;;) {
        a.work.wait(lk, [&] { return a.stop || !a.log.empty(); });
        if (a.log.empty()) {
            if (a.stop) return;
            continue;
        }
        const int32_t len = a.log.front();
        a.log.pop_front();
        a.busy = true;
        lk.unlock();
        apply_observation(len);
        lk.lock();
        a.busy = false;
        if (a.log.empty()) a.idle.notify_all();
    }
}

void Allocator::flush() {
    if (!async_) return;
    std::unique_lock<std::mutex> lk(async_->mu);
    async_->idle.wait(lk, [&] { return async_->log.empty() && !async_->busy; });
}

void Allocator::apply_observation(int32_t len) {
    window_.push(len);
    applied_ += 1;
    if (applied_ % cfg_.refresh == 0) recalibrate();
}

void Allocator::note_observation(int32_t len) {
    observed_ += 1;
    if (async_) {
        {
            std::lock_guard<std::mutex> g(async_->mu);
            async_->log.push_back(len);
        }
        async_->work.notify_one();
    } else {
        apply_observation(len);
    }
}

int32_t Allocator::observe(const int32_t* lengths, int32_t n) {
    if (n < 0 || (n > 0 && !lengths)) return ODMA_ERR_INVALID;
    for (int32_t i = 0; i < n; ++i)
        if (lengths[i] < 0 || lengths[i] > cfg_.max_len) return ODMA_ERR_INVALID;
    for (int32_t i = 0; i < n; ++i) note_observation(lengths[i]);
    return ODMA_OK;
}

int32_t Allocator::drain(int32_t* out, int32_t cap, int32_t* n) {
    if (!n || cap < 0 || (cap > 0 && !out)) return ODMA_ERR_INVALID;
    const int32_t k = static_cast<int32_t>(std::min<size_t>(outbox_.size(), static_cast<size_t>(cap)));
    std::copy(outbox_.begin(), outbox_.begin() + k, out);
    outbox_.erase(outbox_.begin(), outbox_.begin() + k);
    *n = k;
    return ODMA_OK;
}

uint64_t Allocator::epoch() const {
    std::lock_guard<std::mutex> g(bounds_mu_);
    return epoch_;
}

int32_t Allocator::set_buckets(const int32_t* b, int32_t n) {
    if (!b || n < 1 || n > ODMA_MAX_BUCKETS) return ODMA_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        if (b[i] < 1 || b[i] % G_ != 0 || b[i] > cfg_.max_len) return ODMA_ERR_INVALID;
        if (i > 0 && b[i] <= b[i - 1]) return ODMA_ERR_INVALID;
    }
    std::lock_guard<std::mutex> g(bounds_mu_);
    for (int i = 0; i < n; ++i) bounds_[i] = b[i];
    n_bounds_ = n;
    epoch_ += 1;
    return ODMA_OK;
}

int32_t Allocator::get_buckets(int32_t* b, int32_t* n, uint64_t* epoch) const {
    if (!b || !n) return ODMA_ERR_INVALID;
    std::lock_guard<std::mutex> g(bounds_mu_);
    for (int i = 0; i < n_bounds_; ++i) b[i] = static_cast<int32_t>(bounds_[i]);
    *n = n_bounds_;
    if (epoch) *epoch = epoch_;
    return ODMA_OK;
}

const Request* Allocator::find(uint64_t req) const {
    auto it = live_.find(req);
    return it == live_.end() ? nullptr : &it->second;
}

void Allocator::fill(const Request& r, odma_slab* out) const {
    if (!out) return;
    out->base_tok = static_cast<int32_t>(r.base);
    out->cap_tok = static_cast<int32_t>(r.cap);
    out->pool_id = r.pool;
    out->bucket_id = r.bucket;
    out->epoch = epoch();
}

void Allocator::note_safety_peak() {
    const int64_t used = S_ - safety_.free_tokens();
    safety_peak_ = std::max(safety_peak_, used);
}

int32_t Allocator::place_large(int64_t need, int64_t* base, int64_t* cap) {
    int64_t c = cfg_.large_fixed ? cfg_.max_len : ceil_g(need, G_);
    c = std::min<int64_t>(c, cfg_.max_len);
    const int64_t b = safety_.take(c);
    if (b < 0) return ODMA_ERR_NOMEM;
    *base = b;
    *cap = c;
    return ODMA_OK;
}

int32_t Allocator::reserve_large(uint64_t req, int64_t need, odma_slab* out) {
    int64_t base, cap;
    if (place_large(need, &base, &cap) != ODMA_OK) {
        nomem_ += 1;
        return ODMA_ERR_NOMEM;
    }
    Request r;
    r.base = base;
    r.cap = cap;
    r.pool = 1;
    r.bucket = -1;
    r.epoch = epoch();
    live_[req] = r;
    reserved_live_ += cap;
    routed_large_ += 1;
    note_safety_peak();
    fill(r, out);
    return ODMA_OK;
}

int32_t Allocator::reserve(uint64_t req, int64_t predicted, odma_slab* out) {
    if (predicted < 1) return ODMA_ERR_INVALID;
    if (live_.count(req)) return ODMA_ERR_DUP_REQ;
    // one consistent view of the boundaries (a background refresh may replace them at any moment)
    int64_t bnd[ODMA_MAX_BUCKETS];
    int32_t nb;
    uint64_t ep;
    {
        std::lock_guard<std::mutex> g(bounds_mu_);
        nb = n_bounds_;
        for (int i = 0; i < nb; ++i) bnd[i] = bounds_[i];
        ep = epoch_;
    }
    if (predicted > bnd[nb - 1] || predicted > cfg_.max_len)
        return reserve_large(req, std::min<int64_t>(predicted, cfg_.max_len), out);
    int bi = 0;
    while (bnd[bi] < predicted) ++bi;          // first boundary that holds the request
    const int64_t cap = bnd[bi];
    const int64_t base = main_.take(cap);
    if (base < 0) {
        nomem_ += 1;
        return ODMA_ERR_NOMEM;
    }
    Request r;
    r.base = base;
    r.cap = cap;
    r.pool = 0;
    r.bucket = bi;
    r.epoch = ep;
    live_[req] = r;
    reserved_live_ += cap;
    fill(r, out);
    return ODMA_OK;
}

int32_t Allocator::reserve_uncertain(uint64_t req, int64_t l_hat, int64_t u_pm, odma_slab* out) {
    if (l_hat < 1 || u_pm < 0 || u_pm > 1000) return ODMA_ERR_INVALID;
    // ceil(l_hat * (1 + gamma*u)) with gamma and u in thousandths
    const int64_t inflated =
        (l_hat * (1000000 + static_cast<int64_t>(cfg_.gamma_permille) * u_pm) + 999999) / 1000000;
    if (u_pm > cfg_.tau_permille) {
        if (live_.count(req)) return ODMA_ERR_DUP_REQ;
        return reserve_large(req, std::min<int64_t>(inflated, cfg_.max_len), out);
    }
    return reserve(req, inflated, out);
}

int32_t Allocator::ensure(uint64_t req, int64_t need, odma_slab* out, int32_t* migrated,
                          Migration* mig) {
    if (migrated) *migrated = 0;
    auto it = live_.find(req);
    if (it == live_.end()) return ODMA_ERR_UNKNOWN_REQ;
    Request& r = it->second;
    if (need <= r.cap) {
        fill(r, out);
        return ODMA_OK;
    }
    if (need > cfg_.max_len) return ODMA_ERR_OVERFLOW;
    int64_t want = std::max<int64_t>(need, static_cast<int64_t>(cfg_.growth) * r.len);
    want = std::min<int64_t>(want, cfg_.max_len);
    int64_t base, cap;
    if (place_large(want, &base, &cap) != ODMA_OK) {   // allocate first ...
        nomem_ += 1;
        return ODMA_ERR_NOMEM;
    }
    note_safety_peak();                                // both slabs are held at this moment
    if (mig) *mig = Migration{r.base, r.cap, base, cap, r.len};
    (r.pool == 0 ? main_ : safety_).give(r.base, r.cap);   // ... release the old slab last
    reserved_live_ += cap - r.cap;
    r.base = base;
    r.cap = cap;
    r.pool = 1;
    r.bucket = -1;
    r.migrations += 1;
    migrations_ += 1;
    if (migrated) *migrated = 1;
    fill(r, out);
    return ODMA_OK;
}

int32_t Allocator::commit(const uint64_t* reqs, int32_t n, const int32_t* n_new) {
    if (n < 0 || (n > 0 && !reqs)) return ODMA_ERR_INVALID;
    for (int32_t i = 0; i < n; ++i) {
        auto it = live_.find(reqs[i]);
        if (it == live_.end()) return ODMA_ERR_UNKNOWN_REQ;
        const int64_t add = n_new ? n_new[i] : 1;
        if (add < 0 || it->second.len + add > it->second.cap) return ODMA_ERR_OVERFLOW;
    }
    for (int32_t i = 0; i < n; ++i) {
        const int64_t add = n_new ? n_new[i] : 1;
        live_[reqs[i]].len += add;
        used_live_ += add;
    }
    return ODMA_OK;
}

void Allocator::recalibrate() {
    const int64_t n = window_.count();
    int64_t fresh[ODMA_MAX_BUCKETS];
    for (int i = 0; i < cfg_.n_levels; ++i) {
        int64_t rank = (static_cast<int64_t>(cfg_.p_num[i]) * n + cfg_.p_den - 1) / cfg_.p_den;
        rank = std::min(std::max<int64_t>(rank, 1), n);
        const int64_t b = ceil_g(window_.order_statistic(rank), G_);
        fresh[i] = std::min<int64_t>(b, cfg_.max_len);
    }
    std::lock_guard<std::mutex> g(bounds_mu_);
    for (int i = 0; i < cfg_.n_levels; ++i) bounds_[i] = fresh[i];
    n_bounds_ = cfg_.n_levels;
    epoch_ += 1;
}

int32_t Allocator::release(uint64_t req) {
    auto it = live_.find(req);
    if (it == live_.end()) return ODMA_ERR_UNKNOWN_REQ;
    const Request r = it->second;
    live_.erase(it);
    (r.pool == 0 ? main_ : safety_).give(r.base, r.cap);
    reserved_live_ -= r.cap;
    used_live_ -= r.len;
    completed_ += 1;
    sum_len_ += r.len;
    sum_cap_ += r.cap;
    // the realised length: into the window here, or (cluster_observe) only into the outbox, from
    // where the cluster's exchange brings every replica's lengths into every window in one order
    outbox_.push_back(static_cast<int32_t>(r.len));
    if (outbox_.size() > static_cast<size_t>(cfg_.window)) outbox_.erase(outbox_.begin());
    if (!cfg_.cluster_observe) note_observation(static_cast<int32_t>(r.len));
    return ODMA_OK;
}

void Allocator::stats(odma_stats* out) const {
    out->total_tokens = T_;
    out->safety_tokens = S_;
    out->main_tokens = M_;
    out->live = static_cast<int64_t>(live_.size());
    out->reserved_live = reserved_live_;
    out->used_live = used_live_;
    out->completed = completed_;
    out->sum_len_completed = sum_len_;
    out->sum_cap_completed = sum_cap_;
    out->migrations = migrations_;
    out->nomem = nomem_;
    out->routed_large = routed_large_;
    out->safety_live = S_ - safety_.free_tokens();
    out->safety_peak = safety_peak_;
    out->observed = observed_;
    out->epoch = epoch();
}

}  // namespace odma
