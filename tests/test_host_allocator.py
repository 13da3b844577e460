"""The library's C++ allocator against the CPU checker, event by event, bit-exact (no GPU)."""
import numpy as np
import pytest

from conftest import read_golden
from helpers import LockStep, host_pool, lib, oracle_allocator, warm_up
from paper_2512_09427_b200 import workloads as wl


@pytest.mark.parametrize("case", ["1a", "1b"])
def test_config1_matches_the_hand_computed_table(case):
    w = wl.config1(case[-1])
    pool = host_pool(w)
    assert pool.set_buckets(list(w.static_buckets)) == 0
    st = pool.get_stats()
    assert (st["total_tokens"], st["safety_tokens"], st["main_tokens"]) == (1024, 256, 768)
    prefilled = False
    for _, ev, req, arg, base, cap, pl, bucket, mig in [r for r in read_golden("config1_alloc.txt") if r[0] == case]:
        req, arg, base, cap, pl, bucket, mig = map(int, (req, arg, base, cap, pl, bucket, mig))
        if ev == "alloc":
            rc, slab = pool.alloc(req, arg)
            assert rc == 0 and slab[:4] == (base, cap, pl, bucket)
        else:
            if not prefilled:
                assert pool.commit_step(list(range(4)), [int(c) for c in w.context]) == 0
                prefilled = True
            rc, slab, m = pool.ensure_capacity(req, arg)
            assert rc == 0 and m == mig and slab[:4] == (base, cap, pl, bucket)
            assert pool.commit_step([req]) == 0


def test_pool_geometry_golden():
    odma = lib()
    for row in read_golden("pool_geometry.txt"):
        b, nl, hkv, d, s, pct, T, S, M = map(int, row)
        cfg = odma.config_default()
        cfg.safety_pct = pct
        p = odma.Pool(0, b, nl, hkv, d, odma.DTYPE_BF16 if s == 2 else odma.DTYPE_F32, cfg)
        st = p.get_stats()
        assert (st["total_tokens"], st["safety_tokens"], st["main_tokens"]) == (T, S, M)


def test_random_trace_lockstep_including_errors():
    w = wl.scaled(wl.config1("a"), pool_bytes=4096 * 512, window=50, refresh=7)
    ls = LockStep(host_pool(w), oracle_allocator(w))
    assert ls.pool.set_buckets([32, 64, 128, 256]) == ls.oracle.set_buckets([32, 64, 128, 256]) == 0
    rng = np.random.default_rng(3)
    live, nxt = {}, 0
    for _ in range(4000):
        op = rng.random()
        if op < 0.45 or not live:
            if rng.random() < 0.2:
                rc, slab = ls.alloc_uncertain(nxt, int(rng.integers(1, 400)), int(rng.integers(0, 1001)))
                ok = rc == 0
            else:
                ok = ls.alloc(nxt, int(rng.integers(1, 600))) is not None
            if ok:
                live[nxt] = 0
            nxt += 1
        elif op < 0.5:
            r = int(rng.choice(list(live)))
            rc_p, _ = ls.pool.alloc(r, 5)
            rc_o, _ = ls.oracle.reserve(r, 5)
            assert rc_p == rc_o == lib().ERR_DUP_REQ
        elif op < 0.8:
            r = int(rng.choice(list(live)))
            need = live[r] + int(rng.integers(1, 60))
            rc, slab, mig = ls.ensure_rc(r, need)
            if rc == 0:
                ls.commit([r], need - live[r])
                live[r] = need
        else:
            r = int(rng.choice(list(live)))
            ls.free(r)
            del live[r]
    st = ls.check_stats()
    assert st["migrations"] > 10 and st["nomem"] > 0 and st["routed_large"] > 0 and st["epoch"] > 50


def test_config3_batch_with_noisy_predictions():
    w = wl.config3()
    ls = LockStep(host_pool(w), oracle_allocator(w))
    st = ls.check_stats()
    assert (st["total_tokens"], st["safety_tokens"], st["main_tokens"]) == (697536, 69744, 627792)
    warm_up(ls, w.warmup_lengths)
    bounds, epoch = ls.buckets()
    assert epoch == 10 and len(bounds) == 4 and list(bounds) == sorted(bounds)
    for r in range(w.batch):
        assert ls.alloc(r, int(w.predicted[r])) is not None
        ctx = int(w.context[r])
        if ctx > 0:
            ls.ensure(r, ctx)
            ls.commit([r], ctx)
    for r in range(w.batch):
        ls.ensure(r, int(w.context[r]) + 1)
    ls.commit(range(w.batch), 1)
    st = ls.check_stats()
    assert st["used_live"] == int(w.context.sum()) + w.batch
    assert st["migrations"] > 0


@pytest.mark.parametrize("noisy", [False, True])
def test_config4_drift_stream_lockstep(noisy):
    w = wl.config4(n_requests=3000, noisy=noisy)
    ls = LockStep(host_pool(w), oracle_allocator(w))
    assert ls.pool.set_buckets(list(w.static_buckets)) == ls.oracle.set_buckets(list(w.static_buckets)) == 0
    res = wl.run_closed_loop(ls, w.context, w.predicted, w.extra["concurrency"])
    # admissions deferred for lack of memory (ODMA_ERR_NOMEM) are retried after the next completion
    assert res.admitted == 3000
    assert len(res.boundary_log) == 3000 // w.refresh
    st = ls.check_stats()
    assert st["completed"] == 3000
    if noisy:
        assert st["migrations"] > 0
    # after the drift the upper boundaries have moved up with the long mode
    first, last = res.boundary_log[1][1], res.boundary_log[-1][1]
    assert last[-1] > first[-1]


def test_window_turnover_gives_quantiles_of_the_new_distribution():
    # W = 200, R = 100: after 200 completions of the second law nothing of the first remains
    w = wl.scaled(wl.config4(n_requests=10), pool_bytes=1 << 28, window=200, refresh=100)
    pool = host_pool(w)
    lens = np.concatenate([np.full(300, 100), np.arange(1001, 1201)])
    for i, L in enumerate(lens):
        assert pool.alloc(i, int(L))[0] == 0
        assert pool.commit_step([i], [int(L)]) == 0
        assert pool.free(i) == 0
    b, _ = pool.get_buckets()
    want = [int(-(-np.quantile(lens[-200:], q, method="inverted_cdf") // 16) * 16) for q in (0.25, 0.5, 0.75, 1.0)]
    assert list(b) == want


@pytest.mark.parametrize("case,large_fixed", [("LF", 1), ("SP", 0)])
def test_large_bucket_hand_computed_trace(case, large_fixed):
    from test_oracle_allocator import _large_bucket_rows
    odma = lib()
    cfg = odma.config_default()
    cfg.safety_pct, cfg.max_len, cfg.granule, cfg.large_fixed = 50, 512, 16, large_fixed
    pool = odma.Pool(0, 2048 * 512, 1, 1, 64, odma.DTYPE_F32, cfg)
    assert pool.set_buckets([64, 128, 256]) == 0
    for ev, req, arg, rc, slab, mig, live, peak in _large_bucket_rows(case):
        if ev == "alloc":
            got, s = pool.alloc(req, arg)
            assert got == rc and (s[:4] if got == 0 else None) == slab, (ev, req, arg, got, s)
        elif ev == "ensure":
            got, s, m = pool.ensure_capacity(req, arg)
            assert got == rc and (s[:4] if got == 0 else None) == slab, (ev, req, arg, got, s)
            if rc == 0:
                assert m == mig
        elif ev == "grow":
            assert pool.commit_step([req], [arg]) == rc
        else:
            assert pool.free(req) == rc
        st = pool.get_stats()
        assert (st["safety_live"], st["safety_peak"]) == (live, peak), (ev, req, arg, st)


def test_random_trace_lockstep_with_fixed_size_large_bucket():
    # large_fixed = 1: every Large Bucket slab is max_len tokens, on both sides, event by event
    w = wl.scaled(wl.config1("a"), pool_bytes=8192 * 512, safety_pct=50, window=50, refresh=7)
    ls = LockStep(host_pool(w, large_fixed=1), oracle_allocator(w, large_fixed=1))
    assert ls.pool.set_buckets([32, 64, 128]) == ls.oracle.set_buckets([32, 64, 128]) == 0
    rng = np.random.default_rng(11)
    live, nxt, large_caps = {}, 0, set()
    for _ in range(3000):
        op = rng.random()
        if op < 0.45 or not live:
            if rng.random() < 0.3:
                rc, slab = ls.alloc_uncertain(nxt, int(rng.integers(1, 200)), int(rng.integers(0, 1001)))
            else:
                slab = ls.alloc(nxt, int(rng.integers(1, 300)))
                rc = 0 if slab is not None else 2
            if rc == 0:
                live[nxt] = 0
                if slab[2] == 1:
                    large_caps.add(slab[1])
            nxt += 1
        elif op < 0.8:
            r = int(rng.choice(list(live)))
            need = live[r] + int(rng.integers(1, 60))
            rc, slab, mig = ls.ensure_rc(r, need)
            if rc == 0:
                if mig:
                    large_caps.add(slab[1])
                ls.commit([r], need - live[r])
                live[r] = need
        else:
            r = int(rng.choice(list(live)))
            ls.free(r)
            del live[r]
    st = ls.check_stats()
    assert large_caps == {w.max_len}
    assert st["migrations"] > 5 and st["routed_large"] > 5 and st["nomem"] > 0


@pytest.mark.slow
def test_config4_full_drift_stream_lockstep():
    # the whole 10,000-request stream of the drift workload, bit-exact at every event
    w = wl.config4()
    ls = LockStep(host_pool(w), oracle_allocator(w))
    assert ls.pool.set_buckets(list(w.static_buckets)) == ls.oracle.set_buckets(list(w.static_buckets)) == 0
    res = wl.run_closed_loop(ls, w.context, w.predicted, w.extra["concurrency"])
    assert res.admitted == 10000 and len(res.boundary_log) == 10000 // w.refresh
    st = ls.check_stats()
    assert st["completed"] == 10000 and ls.events > 20000
