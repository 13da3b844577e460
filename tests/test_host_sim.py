"""The library's native admission simulator (odma_sim_run) against the checker's plain-Python
one: every counter equal, on the hand-computed traces and on random traces (no GPU)."""
import numpy as np
import pytest

from conftest import read_golden
from helpers import lib
from oracle import oracle as ora
from oracle import sim
from paper_2512_09427_b200 import workloads as wl
from test_oracle_sim import FIELDS, POLICY, trace


def lib_pool(tokens, max_len, safety_pct, buckets, **over):
    odma = lib()
    cfg = odma.config_default()
    cfg.safety_pct, cfg.max_len, cfg.granule = safety_pct, max_len, 16
    for k, v in over.items():
        setattr(cfg, k, v)
    pool = odma.Pool(0, tokens * 512, 1, 1, 64, odma.DTYPE_F32, cfg)
    assert pool.set_buckets(buckets) == 0
    return pool


@pytest.mark.parametrize("row", read_golden("sim_trace.txt"), ids=lambda r: r[0])
def test_hand_computed_traces(row):
    case, policy = row[0], POLICY[row[1]]
    want = dict(zip(FIELDS, map(int, row[3:])))
    reqs, tokens, max_len, safety = trace(case)
    pool = lib_pool(tokens, max_len, safety, [b for b in (16, 32, 64) if b <= max_len])
    got = pool.sim_run(policy, [(r.arrival_ns, r.prompt, r.total, r.predicted, r.u_permille) for r in reqs], 8, 1, 1000, 1000)
    assert got == want


@pytest.mark.parametrize("policy", [sim.STATIC, sim.PAGED, sim.ODMA])
@pytest.mark.parametrize("tight", [False, True])
def test_random_traces_equal_the_checker(policy, tight):
    rng = np.random.default_rng(17 + policy)
    for trial in range(12):
        n = 80
        rows = wl.poisson_trace(1000 + trial, n, rate_per_s=float(rng.choice([2e3, 2e4, 2e5])),
                                law="pareto" if trial % 3 == 0 else "lognormal", max_len=1024,
                                with_uncertainty=trial % 2 == 1)
        rows = [(a, p, min(t, 1024), q, u) for a, p, t, q, u in rows]
        rows = [(a, min(p, t - 1), t, q, u) for a, p, t, q, u in rows]
        tokens = 3072 if tight else 16384
        kw = dict(window=40, refresh=10)
        pool = lib_pool(tokens, 1024, 25, [64, 256, 1024], **kw)
        got = pool.sim_run(policy, rows, 24, 2, 3000, 300)
        alloc = ora.Allocator(tokens * 512, 1, 1, 64, 4, safety_pct=25, max_len=1024, granule=16, **kw)
        assert alloc.set_buckets([64, 256, 1024]) == ora.OK
        want = sim.simulate(policy, tokens, 1024, [sim.SimRequest(*r) for r in rows], max_batch=24, layers=2,
                            base_ns=3000, ps_per_token=300, allocator=alloc if policy == sim.ODMA else None)
        assert got == {k: getattr(want, k) for k in FIELDS}, (policy, tight, trial)
        if policy == sim.ODMA:
            assert pool.get_buckets() == alloc.get_buckets()      # the same lengths were logged in the same order
    assert got["completed"] > 0


def test_rejects_a_pool_with_live_requests_and_bad_traces():
    odma = lib()
    pool = lib_pool(1024, 256, 25, [64, 256])
    assert pool.alloc(5, 10)[0] == 0
    with pytest.raises(odma.OdmaError):
        pool.sim_run(sim.ODMA, [(0, 1, 2, 2, -1)], 4, 1, 1000, 1000)
    pool2 = lib_pool(1024, 256, 25, [64, 256])
    with pytest.raises(odma.OdmaError):
        pool2.sim_run(sim.ODMA, [(10, 1, 2, 2, -1), (5, 1, 2, 2, -1)], 4, 1, 1000, 1000)    # arrivals go back in time
    with pytest.raises(odma.OdmaError):
        pool2.sim_run(sim.ODMA, [(0, 4, 4, 4, -1)], 4, 1, 1000, 1000)                       # nothing to generate
