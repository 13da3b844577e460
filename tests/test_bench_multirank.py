"""Host logic of the multi-GPU benchmark arm, on CPU with gloo (world size 2).

The decode path shards by request with no exchange, so `bench.py --gpus N` runs N independent
replicas; what the ranks share is only the timing reduction (max over ranks) and rank 0's
JSON line.  Both are exercised here without a GPU."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank's timed region took a different time; every rank must end up with the maximum
    mine = [10.0 + 5.0 * rank, float("nan") if rank == 0 else 3.0]
    got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    w, step_layers, copies = bench.pick_workload("config2", rank, 0)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"max": got, "ctx_sum": int(w.context.sum()), "batch": w.batch, "copies": copies}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_per_rank_replicas(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.load(open(tmp_path / f"r{r}.json")) for r in (0, 1))
    assert r0["max"][0] == r1["max"][0] == 15.0
    assert r0["max"][1] == r1["max"][1] == 3.0          # a rank without that measurement does not win
    # replicas: same shape of work per rank (weak scaling), independent seeded inputs
    assert r0["batch"] == r1["batch"] == 64 and r0["ctx_sum"] != r1["ctx_sum"]


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "3"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("configs[1]")
