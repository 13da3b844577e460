"""Pins for the CPU checker's allocator (oracle/odma_oracle.c, part 2).

Hand-computed tables (tests/golden/), numpy's nearest-rank quantile, exact
rational arithmetic, the constants the paper states, and structural invariants
checked from the definition on the raw owner array.
"""
from fractions import Fraction

import numpy as np
import pytest

from conftest import read_golden
from oracle import oracle as ora


def _tiny(**kw):
    args = dict(pool_bytes=1024 * 512, layers=1, kv_heads=1, head_dim=64, elem_bytes=4,
                safety_pct=25, max_len=512, granule=16)
    args.update(kw)
    a = ora.Allocator(**args)
    assert a.set_buckets([64, 128, 256]) == ora.OK
    return a


def test_pool_geometry_golden():
    for row in read_golden("pool_geometry.txt"):
        b, nl, hkv, d, s, pct, T, S, M = map(int, row)
        a = ora.Allocator(b, nl, hkv, d, s, safety_pct=pct)
        assert (a.T, a.S, a.M) == (T, S, M)


@pytest.mark.parametrize("case", ["1a", "1b"])
def test_config1_worked_example(case):
    ctx = [17, 64, 100, 250]
    a = _tiny()
    rows = [r for r in read_golden("config1_alloc.txt") if r[0] == case]
    prefilled = False
    for _, ev, req, arg, base, cap, pool, bucket, mig in rows:
        req, arg, base, cap, pool, bucket, mig = map(int, (req, arg, base, cap, pool, bucket, mig))
        if ev == "alloc":
            if prefilled and req < 4:
                pytest.fail("alloc after prefill only for new requests")
            rc, slab = a.reserve(req, arg)
            assert rc == ora.OK
            assert slab[:4] == (base, cap, pool, bucket)
        else:
            if not prefilled:
                for r, c in enumerate(ctx):
                    assert a.add_len(r, c) == ora.OK
                prefilled = True
            rc, slab, m = a.ensure_capacity(req, arg)
            assert rc == ora.OK and m == mig
            assert slab[:4] == (base, cap, pool, bucket)
            assert a.add_len(req, 1) == ora.OK
    if case == "1b":
        assert a.stats()["migrations"] == 1


def test_bucket_edge_is_inclusive_and_beyond_last_goes_large():
    a = _tiny(pool_bytes=2048 * 512)       # safety region of 512 tokens
    assert a.reserve(1, 64)[1][1] == 64
    assert a.reserve(2, 65)[1][1] == 128
    rc, slab = a.reserve(3, 257)          # beyond the last boundary
    assert rc == ora.OK and slab[2] == 1 and slab[3] == -1 and slab[0] >= a.M
    assert slab[1] == 272                 # ceil16(257)


def test_paper_constants_inflation_and_routing():
    # gamma = 0.2, tau = 0.8 (Section III-B): L' = L(1 + 0.2 u); u > 0.8 -> Large Bucket
    a = _tiny()
    rc, slab = a.reserve_uncertain(1, 100, 500)     # 100 * 1.1 = 110 -> bucket 128
    assert rc == ora.OK and slab[1] == 128 and slab[2] == 0
    rc, slab = a.reserve_uncertain(2, 100, 800)     # u == tau is NOT routed; 116 -> 128
    assert slab[2] == 0 and slab[1] == 128
    rc, slab = a.reserve_uncertain(3, 100, 801)     # routed; ceil(100*1.1602)=117 -> 128 tokens
    assert slab[2] == 1 and slab[3] == -1 and slab[1] == 128 and slab[0] == a.M
    assert a.stats()["routed_large"] == 1


def test_inflation_matches_exact_rational_ceiling():
    rng = np.random.default_rng(0)
    for _ in range(200):
        l_hat = int(rng.integers(1, 400))
        u = int(rng.integers(0, 801))
        exact = Fraction(l_hat) * (1 + Fraction(2, 10) * Fraction(u, 1000))
        want = -((-exact.numerator) // exact.denominator)     # ceil
        a = ora.Allocator(1 << 22, 1, 1, 64, 4, safety_pct=25, max_len=1024)
        a.set_buckets([16 * i for i in range(1, 9)] )
        rc, slab = a.reserve_uncertain(1, l_hat, u)
        assert rc == ora.OK
        if want <= 128:
            assert slab[1] == -(-want // 16) * 16 and slab[2] == 0
        else:
            assert slab[2] == 1 and slab[1] == -(-want // 16) * 16


def _lowest_fit_from_definition(own, lo, hi, cap, G):
    for base in range(lo, hi - cap + 1, G):
        if (own[base:base + cap] == -1).all():
            return base
    return None


def test_placement_is_lowest_address_and_invariants_hold_on_a_random_trace():
    rng = np.random.default_rng(1)
    a = ora.Allocator(4096 * 512, 1, 1, 64, 4, safety_pct=25, max_len=512, granule=16)
    a.set_buckets([32, 64, 128, 256])
    live = {}
    nxt = 0
    for step in range(1500):
        op = rng.random()
        if op < 0.5 or not live:
            P = int(rng.integers(1, 300))
            own = a.owner_array()
            rc, slab = a.reserve(nxt, P)
            if P > 256:
                want = _lowest_fit_from_definition(own, a.M, a.T, -(-P // 16) * 16, 16)
            else:
                cap = [b for b in (32, 64, 128, 256) if b >= P][0]
                want = _lowest_fit_from_definition(own, 0, a.M, cap, 16)
            if want is None:
                assert rc == ora.ERR_NOMEM
            else:
                assert rc == ora.OK and slab[0] == want
                live[nxt] = 0
            nxt += 1
        elif op < 0.8:
            r = int(rng.choice(list(live)))
            own = a.owner_array()
            need = live[r] + int(rng.integers(1, 40))
            rc, slab, mig = a.ensure_capacity(r, need)
            if rc == ora.OK:
                assert slab[1] >= need
                assert a.add_len(r, need - live[r]) == ora.OK
                live[r] = need
            else:
                assert rc in (ora.ERR_NOMEM, ora.ERR_OVERFLOW)
        else:
            r = int(rng.choice(list(live)))
            assert a.release(r) == ora.OK
            del live[r]
        # invariants, from the raw owner array
        own = a.owner_array()
        recs = a.live()
        assert {x[0] for x in recs} == set(live)
        covered = 0
        for rid, base, cap, ln, pool in recs:
            assert base % 16 == 0 and cap % 16 == 0 and cap >= ln
            seg = own[base:base + cap]
            assert (seg == seg[0]).all() and seg[0] != -1          # one owner, contiguous
            if pool == 0:
                assert 0 <= base and base + cap <= a.M
            else:
                assert a.M <= base and base + cap <= a.T
            covered += cap
        assert covered + int((own == -1).sum()) == a.T              # no overlap, nothing lost
    assert a.stats()["migrations"] > 0


def test_free_then_alloc_on_empty_pool_returns_base_zero():
    a = _tiny()
    assert a.reserve(1, 100)[1][0] == 0
    a.release(1)
    assert a.reserve(2, 100)[1][0] == 0


def test_migration_allocates_before_releasing_and_fails_cleanly():
    a = _tiny()                      # safety region 256 tokens
    a.reserve(1, 256)
    a.add_len(1, 256)
    rc, slab, mig = a.ensure_capacity(1, 257)      # wants min(512, max(257, 512)) = 512 > 256
    assert rc == ora.ERR_NOMEM and mig == 0
    assert a.live()[0][1:3] == (0, 256)             # old slab untouched
    assert a.ensure_capacity(1, 513)[0] == ora.ERR_OVERFLOW
    a2 = _tiny()
    a2.reserve(1, 64)
    a2.add_len(1, 64)
    rc, slab, mig = a2.ensure_capacity(1, 65)
    assert (rc, mig) == (ora.OK, 1) and slab[:3] == (768, 128, 1)
    a2.add_len(1, 64)
    rc, slab, mig = a2.ensure_capacity(1, 129)     # second migration, inside the safety region
    # the old safety slab [768,896) is still held while the new one is placed
    assert rc == ora.ERR_NOMEM or slab[0] >= 896


def test_errors():
    a = _tiny()
    assert a.reserve(1, 0)[0] == ora.ERR_INVALID
    assert a.reserve(1, 10)[0] == ora.OK
    assert a.reserve(1, 10)[0] == ora.ERR_DUP_REQ
    assert a.release(2) == ora.ERR_UNKNOWN_REQ
    assert a.ensure_capacity(2, 5)[0] == ora.ERR_UNKNOWN_REQ
    assert a.add_len(1, 65) == ora.ERR_OVERFLOW
    assert a.set_buckets([64, 64]) == ora.ERR_INVALID
    assert a.set_buckets([60, 128]) == ora.ERR_INVALID
    assert a.set_buckets([64, 1024]) == ora.ERR_INVALID
    # main region exhausted: ordinary requests do not spill into the safety pool
    b = _tiny()
    for i in range(3):
        assert b.reserve(i, 256)[0] == ora.OK
    assert b.reserve(9, 200)[0] == ora.ERR_NOMEM
    assert b.stats()["nomem"] == 1


@pytest.mark.parametrize("p_num,p_den", [((1, 2, 3, 4), 4), ((50, 80, 95, 99), 100)])
def test_boundaries_are_library_nearest_rank_quantiles(p_num, p_den):
    # defaults of Section III-C: 4 buckets, window 10,000, refresh every 1,000
    W, R = 10000, 1000
    rng = np.random.default_rng(2)
    lens = np.clip(np.rint(np.exp(rng.normal(6, 0.8, size=12500))), 1, 4000).astype(int)
    a = ora.Allocator(1 << 30, 1, 1, 64, 4, safety_pct=10, max_len=4096, p_num=p_num, p_den=p_den)
    a.set_buckets([4096])
    _, e0 = a.get_buckets()
    for i, L in enumerate(lens):
        assert a.reserve(i, int(L))[0] == ora.OK
        assert a.add_len(i, int(L)) == ora.OK
        assert a.release(i) == ora.OK
        b, e = a.get_buckets()
        seen = i + 1
        if seen % R == 0:
            window = lens[max(0, seen - W):seen]
            want = []
            for pn in p_num:
                qv = np.quantile(window, pn / p_den, method="inverted_cdf")
                want.append(min(4096, -(-int(qv) // 16) * 16))
            assert list(b) == want, (seen, b, want)
            assert e == e0 + seen // R
        else:
            assert e == e0 + seen // R        # no change between refreshes


def test_boundary_update_leaves_live_slabs_alone_and_applies_to_new_requests():
    a = ora.Allocator(1 << 24, 1, 1, 64, 4, safety_pct=10, max_len=1024, window=100, refresh=10)
    a.set_buckets([512, 1024])
    rc, before = a.reserve(1000, 300)
    assert before[1] == 512
    for i in range(10):                      # ten completions of length 40 -> boundaries {48,...}
        a.reserve(i, 40)
        a.add_len(i, 40)
        a.release(i)
    b, _ = a.get_buckets()
    assert list(b) == [48, 48, 48, 48]
    assert [x for x in a.live() if x[0] == 1000][0][1:3] == (before[0], 512)
    rc, slab = a.reserve(1001, 40)
    assert slab[1] == 48 and slab[3] == 0     # duplicates: first matching boundary
    rc, slab = a.reserve(1002, 300)           # now beyond the last boundary -> Large Bucket
    assert slab[2] == 1


def test_utilisation_formula_counts_capacity_at_completion():
    a = _tiny()
    a.reserve(1, 64); a.add_len(1, 50); a.release(1)       # 50 / 64
    a.reserve(2, 64); a.add_len(2, 64)
    a.ensure_capacity(2, 65); a.add_len(2, 1); a.release(2)  # 65 / 128 (capacity held at completion)
    s = a.stats()
    assert (s["sum_len_completed"], s["sum_cap_completed"]) == (115, 192)


def _large_bucket_rows(case):
    """Rows of tests/golden/large_bucket.txt for one case: (event, req, arg, expected fields)."""
    for row in read_golden("large_bucket.txt"):
        if row[0] != case:
            continue
        row = [x for x in row if x != "|"]
        ev, req, arg, rc = row[1], int(row[2]), int(row[3]), int(row[4])
        slab = None if row[5] == "-" else tuple(int(x) for x in row[5:9])
        mig = None if row[9] == "-" else int(row[9])
        yield ev, req, arg, rc, slab, mig, int(row[10]), int(row[11])


@pytest.mark.parametrize("case,large_fixed", [("LF", 1), ("SP", 0)])
def test_large_bucket_hand_computed_trace(case, large_fixed):
    # Section III-D / IV-C: Large Bucket slab sizes (one worst-case size when large_fixed),
    # allocate-then-release order of a migration, and what safety_live / safety_peak count
    a = ora.Allocator(2048 * 512, 1, 1, 64, 4, safety_pct=50, max_len=512, granule=16, large_fixed=large_fixed)
    assert (a.T, a.S, a.M) == (2048, 1024, 1024)
    assert a.set_buckets([64, 128, 256]) == ora.OK
    for ev, req, arg, rc, slab, mig, live, peak in _large_bucket_rows(case):
        if ev == "alloc":
            got, s = a.reserve(req, arg)
            assert got == rc and (s[:4] if s else None) == slab, (ev, req, arg, got, s)
        elif ev == "ensure":
            got, s, m = a.ensure_capacity(req, arg)
            assert got == rc and (s[:4] if s else None) == slab, (ev, req, arg, got, s)
            if rc == ora.OK:
                assert m == mig
        elif ev == "grow":
            assert a.add_len(req, arg) == rc
        else:
            assert a.release(req) == rc
        st = a.stats()
        assert (st["safety_live"], st["safety_peak"]) == (live, peak), (ev, req, arg, st)
