"""Pins for the checker's admission simulator (oracle/sim.py): hand-computed traces
(tests/golden/sim_trace.txt) and conservation properties on random traces."""
import numpy as np
import pytest

from conftest import read_golden
from oracle import oracle as ora
from oracle import sim

FIELDS = ["completed", "failed", "tokens_out", "tokens_lost", "steps", "makespan_ns", "sum_actual", "sum_reserved",
          "conc_time", "reserved_time", "used_time", "migrations", "preemptions", "stalls", "deferred"]
POLICY = {"static": sim.STATIC, "paged": sim.PAGED, "odma": sim.ODMA}


def trace(case):
    if case.startswith("A_"):
        pred1 = 16 if case == "A_ODMA_b" else 20
        reqs = [sim.SimRequest(0, 4, 6, 6), sim.SimRequest(0, 15, 18, pred1), sim.SimRequest(2500, 8, 9, 9)]
        return reqs, 128, 64, 25
    reqs = [sim.SimRequest(0, 16, 18, 18), sim.SimRequest(0, 15, 17, 17)]
    return reqs, 32, 32, 0


def tiny_allocator(tokens, max_len, safety_pct):
    a = ora.Allocator(tokens * 512, 1, 1, 64, 4, safety_pct=safety_pct, max_len=max_len, granule=16)
    assert a.T == tokens
    assert a.set_buckets([b for b in (16, 32, 64) if b <= max_len]) == ora.OK
    return a


@pytest.mark.parametrize("row", read_golden("sim_trace.txt"), ids=lambda r: r[0])
def test_hand_computed_traces(row):
    case, policy = row[0], POLICY[row[1]]
    want = dict(zip(FIELDS, map(int, row[3:])))
    reqs, tokens, max_len, safety = trace(case)
    alloc = tiny_allocator(tokens, max_len, safety) if policy == sim.ODMA else None
    res = sim.simulate(policy, tokens, max_len, reqs, max_batch=8, layers=1, base_ns=1000, ps_per_token=1000,
                       allocator=alloc)
    got = {k: getattr(res, k) for k in FIELDS}
    assert got == want


@pytest.mark.parametrize("policy", [sim.STATIC, sim.PAGED, sim.ODMA])
def test_conservation_on_random_traces(policy):
    rng = np.random.default_rng(4 + policy)
    for trial in range(20):
        n = 60
        total = np.clip(np.rint(np.exp(rng.normal(4.5, 0.8, size=n))), 4, 500).astype(int)
        prompt = np.maximum(1, total // 3)
        pred = np.maximum(1, np.rint(total * np.exp(rng.normal(0, 0.3, size=n)))).astype(int)
        arr = np.cumsum(rng.exponential(20000, size=n)).astype(int)
        reqs = [sim.SimRequest(int(a), int(p), int(t), int(q), int(rng.integers(0, 1001)) if trial % 2 else -1)
                for a, p, t, q in zip(arr, prompt, total, pred)]
        tokens = 2048
        alloc = None
        if policy == sim.ODMA:
            alloc = ora.Allocator(tokens * 512, 1, 1, 64, 4, safety_pct=25, max_len=512, granule=16)
            assert alloc.set_buckets([32, 64, 128, 512]) == ora.OK
        res = sim.simulate(policy, tokens, 512, reqs, max_batch=16, layers=2, base_ns=3000, ps_per_token=300000,
                           allocator=alloc)
        assert res.completed + res.failed == n
        done = [e for e in res.log if e[0] == "done"]
        assert res.sum_actual == sum(reqs[e[2]].total for e in done)
        # every completed request generated total - prompt tokens; preempted runs add the lost ones
        assert res.tokens_out == sum(reqs[e[2]].total - reqs[e[2]].prompt for e in done) + res.tokens_lost
        assert res.sum_reserved >= res.sum_actual and res.reserved_time >= res.used_time
        assert res.conc_time <= 16 * res.makespan_ns and res.makespan_ns >= int(arr[-1])
        if policy == sim.STATIC:
            assert res.sum_reserved == 512 * res.completed and res.migrations == 0
        if policy == sim.PAGED:
            assert res.sum_reserved == sum(-(-reqs[e[2]].total // 16) * 16 for e in done)
        if policy == sim.ODMA:
            assert alloc.stats()["live"] == 0 and alloc.stats()["migrations"] == res.migrations
