"""Boundary refresh off the critical path (background thread) and across replicas (observation
exchange): at quiescence both must hold exactly the boundaries the checker derives from the same
sequence of realised lengths."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from helpers import LockStep, host_pool, oracle_allocator
from paper_2512_09427_b200 import workloads as wl


def small_workload():
    ctx = np.zeros(1, dtype=np.int64)
    return wl.Workload(name="recal", seed=5, layers=1, q_heads=4, kv_heads=2, head_dim=64, dtype=torch.bfloat16,
                       pool_bytes=1 << 26, safety_pct=10, max_len=4096, context=ctx, predicted=ctx + 1, window=400,
                       refresh=50)


def lengths(seed, n):
    rng = np.random.default_rng(seed)
    return np.clip(np.round(np.exp(rng.normal(np.log(300), 0.9, size=n))), 1, 4096).astype(np.int64)


def replay(alloc_like, lens, first=1 << 30):
    for i, L in enumerate(lens):
        r = first + i
        rc = alloc_like.alloc(r, int(L))
        assert rc is not None
        alloc_like.commit([r], int(L))
        alloc_like.free(r)


def test_async_refresh_matches_the_checker_at_quiescence():
    w = small_workload()
    pool = host_pool(w, async_recal=1)
    orc = oracle_allocator(w)
    lens = lengths(1, 1234)
    for i, L in enumerate(lens):
        r = 1000 + i
        assert pool.alloc(r, int(L))[0] == 0
        assert pool.commit_step([r], [int(L)]) == 0
        assert pool.free(r) == 0
        assert orc.reserve(r, int(L))[0] == 0
        assert orc.add_len(r, int(L)) == 0
        assert orc.release(r) == 0
    pool.recal_flush()
    assert pool.get_buckets() == orc.get_buckets()
    assert pool.get_stats()["observed"] == len(lens)


def test_async_refresh_in_lock_step_when_flushed_before_every_admission():
    """With a flush before each admission the background path is indistinguishable from the
    synchronous one: slabs, boundaries and epochs agree with the checker at every call."""
    w = small_workload()
    pool = host_pool(w, async_recal=1)
    ls = LockStep(pool, oracle_allocator(w))
    lens = lengths(2, 400)
    live = []
    for i, L in enumerate(lens):
        pool.recal_flush()
        r = 5000 + i
        assert ls.alloc(r, int(L)) is not None
        ls.commit([r], int(L))
        live.append(r)
        if len(live) > 7:
            ls.pool.recal_flush()
            rc_o = ls.oracle.release(live[0]); rc_p = ls.pool.free(live[0])
            assert rc_o == rc_p == 0
            live.pop(0)
    pool.recal_flush()
    assert pool.get_buckets() == ls.oracle.get_buckets()


def test_async_thread_stops_with_the_pool_and_bad_flags_are_refused():
    from paper_2512_09427_b200 import odma
    w = small_workload()
    for _ in range(20):                       # create, log, destroy at once: the destructor joins the thread
        pool = host_pool(w, async_recal=1)
        assert pool.alloc(1, 100)[0] == 0 and pool.commit_step([1], [100]) == 0 and pool.free(1) == 0
        pool.destroy()
    with pytest.raises(odma.OdmaError):
        host_pool(w, async_recal=2)
    with pytest.raises(odma.OdmaError):
        host_pool(w, cluster_observe=-1)
    for bad in (-1, 3):                                 # the decode kernel's read-out order: auto, late, at once
        with pytest.raises(odma.OdmaError):
            host_pool(w, readout=bad)
    for good in (odma.READOUT_AUTO, odma.READOUT_LATE, odma.READOUT_AT_ONCE):
        host_pool(w, readout=good).destroy()


def test_observe_and_drain_single_process():
    from paper_2512_09427_b200.cluster import ClusterManager
    w = small_workload()
    pool = host_pool(w, cluster_observe=1)
    orc = oracle_allocator(w)
    lens = lengths(3, 180)
    for i, L in enumerate(lens):
        assert pool.alloc(i, int(L))[0] == 0 and pool.commit_step([i], [int(L)]) == 0 and pool.free(i) == 0
    # nothing has entered the window yet: one bucket of max_len, epoch 0
    assert pool.get_buckets() == ((4096,), 0)
    cm = ClusterManager(pool)
    merged = cm.sync()
    assert merged == [int(x) for x in lens] and pool.drain_observations() == []
    for i, L in enumerate(lens):
        assert orc.reserve(i, int(L))[0] == 0 and orc.add_len(i, int(L)) == 0 and orc.release(i) == 0
    assert pool.get_buckets() == orc.get_buckets()
    # bad observations are refused as a whole
    from paper_2512_09427_b200 import odma
    with pytest.raises(odma.OdmaError):
        pool.observe([10, -1])
    with pytest.raises(odma.OdmaError):
        pool.observe([5000])


_RANK_SCRIPT = r"""
import os, sys, json
import numpy as np, torch, torch.distributed as dist
sys.path.insert(0, os.path.join(os.environ["REPO"], "tests")); sys.path.insert(0, os.environ["REPO"])
from helpers import host_pool, oracle_allocator
from test_recal_async_cluster import small_workload, lengths
from paper_2512_09427_b200.cluster import ClusterManager
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = small_workload()
pool = host_pool(w, cluster_observe=1, async_recal=rank % 2)      # one replica refreshes in the background
cm = ClusterManager(pool)
per_round = [37, 80, 55]
mine = lengths(100 + rank, sum(per_round))
orc = oracle_allocator(w)
k, rid = 0, 0
for n in per_round:
    for L in mine[k:k + n]:
        assert pool.alloc(rid, int(L))[0] == 0 and pool.commit_step([rid], [int(L)]) == 0 and pool.free(rid) == 0
        rid += 1
    merged = cm.sync()
    # the checker sees what every replica saw: rank 0's lengths of the round, then rank 1's
    want = [int(x) for r in range(world) for x in lengths(100 + r, sum(per_round))[k:k + n]]
    assert merged == want, (rank, len(merged), len(want))
    for L in want:
        assert orc.reserve(1 << 20, int(L))[0] == 0 and orc.add_len(1 << 20, int(L)) == 0 and orc.release(1 << 20) == 0
    assert pool.get_buckets() == orc.get_buckets(), (rank, pool.get_buckets(), orc.get_buckets())
    k += n
out = [None] * world
dist.all_gather_object(out, pool.get_buckets())
assert all(o == out[0] for o in out)
if rank == 0:
    print("OK", json.dumps(out[0]))
dist.destroy_process_group()
"""


def test_two_replicas_derive_the_same_boundaries(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT)
    repo = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, REPO=repo)
    port = 29500 + os.getpid() % 2000
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                         env=env, capture_output=True, text=True, timeout=280)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-2000:]
    assert "OK" in res.stdout
