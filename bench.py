"""Decode-step benchmark of the slab-KV attention path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2|config3|config5]
                    [--impl ours|reference]

One step = one pass of the whole device path over one batch: per-step tables (host split plan
+ one small copy), KV append of one new token per request, split decode attention over every
request's slab and the log-sum-exp combine, for the layers the workload steps through.
Prints one JSON line (rank 0).  `value` = decode tokens/s with every input resident in HBM;
`e2e` = the same step from pinned HOST buffers through odma_decode_step_host, copies inside
the timed region; `roofline` = the decode kernel's algorithmic KV bytes over its CUDA-event
time against the measured copy bandwidth; `cpu_baseline` = the fp64 CPU checker timed on the
host cores (a reported baseline).  `--impl reference` times the CPU checker alone.

Multi-GPU (torchrun, one rank per GPU): independent replicas of the same step, no collective
on the data path; timing is barrier + synchronize on both sides, max over ranks.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2512_09427_b200 import workloads as wl  # noqa: E402

METRIC = "decode tokens/s (slab-KV attention path: append + split decode + combine)"
UNIT = "tokens/s"
L2_BYTES = 126 * 2**20
FALLBACK_HBM_GBS = 6650.0
DECODE_KERNELS = {"auto": 0, "tcgen05": 1, "mma_sync": 2}
MIN_TIMED_SECONDS = 0.5      # the K-step region is repeated until this much device time has been timed
MIN_REGION_STEPS = 256       # a timed region is a whole multiple of K steps, at least this many (an event between two
                             # launches makes the second wait for the first: one bracket per 20 steps costs 0.9 us a step)


# ---------------------------------------------------------------------------------------------
# workload set-up through the C ABI (no checker code on this path)
# ---------------------------------------------------------------------------------------------

def pick_workload(name: str, rank: int = 0, copies_override: int = 0, layers_override: int = 0, kv_dtype: str = "bf16"):
    """Returns (workload, layers stepped per step, number of rotating KV copies).

    config2 is one layer; the pool is given several `layers`, each an independent copy of the
    single-layer cache, and consecutive steps rotate over them so that no step finds its KV in
    L2 (one copy is ~90 MB, L2 is 126 MB).  config3/config5 step through all their layers,
    which together are far larger than L2; `layers_override` keeps only that many of them (same
    per-layer sizes, pool shrunk in proportion) for captures that must stay small.
    `kv_dtype` "e4m3": the same requests on 8-bit slabs (half the KV bytes per token)."""
    seed_off = 1000 * rank
    esz = 1 if kv_dtype == "e4m3" else 2
    if name == "config2":
        base = wl.config2(seed=950902 + seed_off)
        kv_bytes = int((base.context + 1).sum()) * 2 * base.kv_heads * base.head_dim * esz
        copies = copies_override or max(4, -(-3 * L2_BYTES // kv_bytes))
        w = wl.config2(layers=copies, seed=950902 + seed_off)
        step_layers = 1
    elif name == "config3":
        w = wl.config3(seed=950903 + seed_off)
        copies, step_layers = 1, w.layers
    elif name == "config5":
        w = wl.config5(seed=950905 + seed_off)
        copies, step_layers = 1, w.layers
    else:
        raise SystemExit(f"unknown workload {name}")
    if layers_override and name != "config2" and layers_override < w.layers:
        w = wl.scaled(w, layers=layers_override, pool_bytes=w.pool_bytes * layers_override // w.layers)
        step_layers = layers_override
    if kv_dtype == "e4m3":
        w = wl.with_e4m3(w)
    return w, step_layers, copies


class _HostLoop:
    """The library's allocator (a bookkeeping-only pool: no device memory) behind the face
    workloads.run_closed_loop drives."""

    def __init__(self, pool, odma):
        self.pool, self.odma = pool, odma

    def alloc(self, req, predicted):
        rc, slab = self.pool.alloc(req, predicted)
        return slab[:4] if rc == self.odma.OK else None

    def ensure(self, req, need):
        rc, slab, mig = self.pool.ensure_capacity(req, need)
        if rc == self.odma.ERR_NOMEM:
            return None
        assert rc == self.odma.OK, rc
        return slab[:4], mig

    def commit(self, reqs, n_new):
        reqs = list(reqs)
        assert self.pool.commit_step(reqs, [n_new] * len(reqs)) == 0

    def free(self, req):
        assert self.pool.free(req) == 0

    def buckets(self):
        return self.pool.get_buckets()


def config4_drift(rank: int = 0):
    """Config 4 on the host: the whole 10,000-request drift stream through the library's
    allocator (closed loop of 128 live requests).  Returns the allocator's statistics and two
    snapshots of the live batch, one from each half of the stream, as workloads for the GPU."""
    from paper_2512_09427_b200 import odma
    w = wl.config4(seed=950904 + 1000 * rank)
    cfg = odma.config_default()
    cfg.safety_pct, cfg.max_len, cfg.granule, cfg.window, cfg.refresh = w.safety_pct, w.max_len, w.granule, w.window, w.refresh
    pool = odma.Pool(0, w.pool_bytes, w.layers, w.kv_heads, w.head_dim, odma.DTYPE_BF16, cfg)
    assert pool.set_buckets(list(w.static_buckets)) == 0
    snaps = {}

    def on_epoch(epoch, live, lens):
        snaps[epoch] = ([int(r) for r in live], np.asarray(lens, dtype=np.int64).copy(), pool.get_buckets()[0])

    res = wl.run_closed_loop(_HostLoop(pool, odma), w.context, w.predicted, w.extra["concurrency"], on_epoch=on_epoch)
    st = pool.get_stats()
    n_req = int(w.context.shape[0])
    stats = {"requests": n_req, "completed": st["completed"], "utilisation": st["sum_len_completed"] / max(st["sum_cap_completed"], 1),
             "static_utilisation": float(w.context.sum()) / (n_req * w.max_len), "migrations": st["migrations"],
             "migration_rate": st["migrations"] / n_req, "deferred_admissions": res.deferred, "preempted": res.preempted,
             "large_bucket_peak_tokens": st["safety_peak"], "recalibrations": len(res.boundary_log),
             "boundaries_first_half": list(res.boundary_log[len(res.boundary_log) // 4][1]),
             "boundaries_second_half": list(res.boundary_log[-2][1])}
    epochs = sorted(snaps)
    halves = []
    for name, e in (("first half (lognormal, median 256)", epochs[len(epochs) // 4]),
                    ("second half (70% median 128 / 30% median 4096)", epochs[-2])):
        live, lens, bounds = snaps[e]
        total = w.context[np.asarray(live)]
        ctx = np.maximum(lens - 1, 1)
        tokens = int(sum(min(b for b in bounds if b >= t) if t <= bounds[-1] else -(-int(t) // 16) * 16 for t in total) / 0.85) + 4096
        halves.append((name, e, wl.Workload(
            name="config4", seed=w.seed + e, layers=1, q_heads=w.q_heads, kv_heads=w.kv_heads, head_dim=w.head_dim,
            dtype=w.dtype, pool_bytes=tokens * 2 * w.kv_heads * w.head_dim * 2, safety_pct=15, max_len=w.max_len,
            context=ctx, predicted=np.maximum(total, ctx + 1), static_buckets=tuple(sorted(set(int(b) for b in bounds))))))
    return stats, halves


READOUT = 0          # --readout: the tcgen05 kernel's read-out order (0 = the library picks per launch)


class SlabDecode:
    """A device pool filled with the workload's KV, plus the step's input buffers."""

    def __init__(self, w: wl.Workload, step_layers: int, device: torch.device, plan_ctas: int = 0,
                 fused: int = 1, decode_kernel: int = 0, chain_launches: int = 1, mem=None):
        from paper_2512_09427_b200 import odma
        self.odma, self.w, self.dev, self.step_layers = odma, w, device, step_layers
        self.dt = (odma.DTYPE_FP8_E4M3 if w.kv_dtype == "e4m3" else
                   odma.DTYPE_BF16 if w.dtype == torch.bfloat16 else odma.DTYPE_F32)
        cfg = odma.config_default()
        cfg.safety_pct, cfg.max_len, cfg.granule = w.safety_pct, w.max_len, w.granule
        cfg.window, cfg.refresh = w.window, w.refresh
        pn, pd = w.quantiles
        cfg.n_levels = len(pn)
        for i, x in enumerate(pn):
            cfg.p_num[i] = x
        cfg.p_den = pd
        cfg.max_batch = max(1024, w.batch)
        cfg.plan_ctas = plan_ctas
        cfg.fused_combine = fused
        cfg.decode_kernel = decode_kernel
        cfg.chain_launches = chain_launches
        cfg.readout = READOUT
        self.pool_cfg = cfg
        # `mem`: the device memory of another SlabDecode of the same workload (a second pool over the
        # same, already filled bytes: the allocator is deterministic, so the slabs coincide)
        self.mem = mem if mem is not None else torch.zeros(w.pool_bytes, dtype=torch.uint8, device=device)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.pool = odma.Pool(self.mem.data_ptr(), w.pool_bytes, w.layers, w.kv_heads, w.head_dim,
                              self.dt, cfg)
        if w.kv_dtype == "e4m3":
            self.pool.set_kv_scales(*wl.e4m3_scales(w.layers))
        self.reqs = list(range(w.batch))
        self.reqs_c = (C.c_uint64 * w.batch)(*self.reqs)
        self.zeros_c = (C.c_int32 * w.batch)()
        self.migrations_at_fill = 0
        self._ptrs = {}

    def learn_boundaries(self):
        """Static ladder, or boundaries learned from the warm-up window of realised lengths."""
        w, pool = self.w, self.pool
        if w.static_buckets:
            assert pool.set_buckets(list(w.static_buckets)) == 0
        if w.warmup_lengths is not None:
            for i, L in enumerate(w.warmup_lengths):
                r = (1 << 40) + i
                rc, _ = pool.alloc(r, int(L))
                assert rc == 0, rc
                assert pool.commit_step([r], [int(L)]) == 0
                assert pool.free(r) == 0
        return pool.get_buckets()

    def admit_and_fill(self, fill: bool = True):
        """Reserve every request's slab and write its context tokens (seeded N(0,1)) on all layers
        (`fill` False: the memory already holds them, only the bookkeeping is done)."""
        w, pool, odma = self.w, self.pool, self.odma
        for r in self.reqs:
            rc, _ = pool.alloc(r, int(w.predicted[r]))
            assert rc == odma.OK, ("alloc", r, rc)
            rc, _, _ = pool.ensure_capacity(r, int(w.context[r]) + 1, self.stream)
            assert rc == odma.OK, ("ensure", r, rc)
        if not fill:
            assert pool.commit_step(self.reqs, [int(c) for c in w.context]) == 0
            torch.cuda.synchronize()
            return
        table = torch.empty(pool.tables_bytes(w.batch), dtype=torch.uint8, device=self.dev)
        ctx = [int(c) for c in w.context]
        t = pool.build_tables(self.reqs, table.data_ptr(), table.numel(), self.stream, ctx)
        chunk = max(1, (1 << 26) // (w.kv_heads * w.head_dim))      # tokens per generated piece
        for layer in range(w.layers):
            for kind, name in ((wl.KIND_K, "k"), (wl.KIND_V, "v")):
                pieces = [wl.kv_rows(w.seed, layer, r, kind, t0, min(t0 + chunk, c), w.kv_heads,
                                     w.head_dim, w.dtype, self.dev)
                          for r, c in zip(self.reqs, ctx) for t0 in range(0, c, chunk)]
                if name == "k":
                    k_all = torch.cat(pieces)
                else:
                    v_all = torch.cat(pieces)
            pool.append_kv(layer, t, k_all.data_ptr(), v_all.data_ptr(), self.stream)
            torch.cuda.synchronize()
            del k_all, v_all, pieces
        assert pool.commit_step(self.reqs, ctx) == 0
        self.migrations_at_fill = pool.get_stats()["migrations"]

    def make_inputs(self, pinned: bool = False):
        """Per layer: q [n,Hq,D] and the new token's K/V rows [n,Hkv,D] (seeded), and out."""
        w = self.w
        q = torch.stack([torch.stack([wl.q_rows(w.seed, l, r, 0, w.q_heads, w.head_dim, w.dtype, self.dev)
                                      for r in self.reqs]) for l in range(w.layers)]).contiguous()
        kn = torch.stack([torch.cat([wl.kv_rows(w.seed, l, r, wl.KIND_K, int(w.context[r]), int(w.context[r]) + 1,
                                                w.kv_heads, w.head_dim, w.dtype, self.dev) for r in self.reqs])
                          for l in range(w.layers)]).contiguous()
        vn = torch.stack([torch.cat([wl.kv_rows(w.seed, l, r, wl.KIND_V, int(w.context[r]), int(w.context[r]) + 1,
                                                w.kv_heads, w.head_dim, w.dtype, self.dev) for r in self.reqs])
                          for l in range(w.layers)]).contiguous()
        out = torch.zeros_like(q)
        if pinned:
            return tuple(x.cpu().pin_memory() for x in (q, kn, vn, out))
        return q, kn, vn, out

    def step(self, i: int, q, kn, vn, out, tables=None):
        """Step i from device buffers: the layers it touches, one C call, then the length commit."""
        L = self.step_layers
        l0 = (i * L) % self.w.layers
        key = (q.data_ptr(), l0)
        ptrs = self._ptrs.get(key)
        if ptrs is None:                         # tensor indexing costs microseconds: do it once
            ptrs = self._ptrs[key] = (q[l0].data_ptr(), kn[l0].data_ptr(), vn[l0].data_ptr(), out[l0].data_ptr())
        self.pool.decode_step(l0, L, self.w.q_heads, self.reqs_c, ptrs[0], ptrs[1], ptrs[2], ptrs[3], 0,
                              self.stream, tables)
        self.commit_none()

    def commit_none(self):
        """Every timed step repeats the SAME decode step (token `context` appended, context+1
        keys attended), so that K steps measure one workload rather than a growing one: the
        host-side length commit runs, with zero growth."""
        rc = self.odma._lib.odma_commit_step(self.pool._h, self.reqs_c, self.w.batch, self.zeros_c)
        assert rc == 0, rc

    def step_host(self, i: int, hq, hkn, hvn, hout):
        """Step i from pinned host buffers; the result is on the host when this returns."""
        L = self.step_layers
        l0 = (i * L) % self.w.layers
        for l in range(l0, l0 + L):
            key = (hq.data_ptr(), l)
            ptrs = self._ptrs.get(key)
            if ptrs is None:                     # tensor indexing costs microseconds: do it once
                ptrs = self._ptrs[key] = (hq[l].data_ptr(), hkn[l].data_ptr(), hvn[l].data_ptr(), hout[l].data_ptr())
            self.pool.decode_step_host(l, self.w.q_heads, self.reqs_c, ptrs[0], ptrs[1], ptrs[2], ptrs[3], self.stream)
        torch.cuda.current_stream().synchronize()
        self.commit_none()


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

_CLOCK_FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
                 "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                 "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


class ClockSampler:
    """nvidia-smi in a child process, one CSV line every 50 ms, read-only queries."""

    def __init__(self, gpu_index: int):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.f = open(self.path, "w")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={_CLOCK_FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        self.windows = []

    def mark(self, t0: float, t1: float):
        self.windows.append((t0, t1))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.f.close()
        from datetime import datetime
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 10:
                continue
            try:
                ts = datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                mhz, mx = float(parts[2]), float(parts[3])
            except ValueError:
                continue
            if not any(a - 0.05 <= ts <= b + 0.05 for a, b in self.windows):
                continue
            sm.append(mhz)
            smax.append(mx)
            for nm, val in zip(names, parts[6:10]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        try:
            os.unlink(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# CPU checker legs (the only place this file touches oracle/)
# ---------------------------------------------------------------------------------------------

def _host_batch(w: wl.Workload, reqs, layer=0):
    """(q, K list, V list) of the decode step of `reqs` on one layer, generated on the CPU."""
    q = torch.stack([wl.q_rows(w.seed, layer, r, 0, w.q_heads, w.head_dim, w.dtype) for r in reqs])
    Ks = [wl.kv_rows(w.seed, layer, r, wl.KIND_K, 0, int(w.context[r]) + 1, w.kv_heads, w.head_dim, w.dtype) for r in reqs]
    Vs = [wl.kv_rows(w.seed, layer, r, wl.KIND_V, 0, int(w.context[r]) + 1, w.kv_heads, w.head_dim, w.dtype) for r in reqs]
    return q, Ks, Vs


def checker_sample(w: wl.Workload, step_layers: int, budget_s: float):
    """Times the CPU checker on a bounded sample of the step: the first m requests of the
    batch on one layer (requests are i.i.d., so any prefix has the batch's length law), with m
    chosen from a one-request probe so that the sample takes about `budget_s` seconds."""
    from oracle import oracle as ora
    ora.build()
    code = ora.dtype_code(w.dtype)
    q, Ks, Vs = _host_batch(w, [0])
    t0 = time.perf_counter()
    _, _, threads = ora.decode_attention(q, Ks, Vs, w.q_heads, w.kv_heads, w.head_dim, code)
    probe = max(time.perf_counter() - t0, 1e-6)
    per_tok = probe / float(w.context[0] + 1)             # one request runs on one thread
    total = np.cumsum(w.context + 1)
    cores = os.cpu_count() or 1
    m = int(np.searchsorted(total * per_tok / min(cores, w.batch), budget_s) + 1)
    m = max(1, min(w.batch, m))
    return m, threads


def checker_time_step(w: wl.Workload, m: int, step_layers: int):
    """One timed pass of the CPU checker over the first m requests (one layer); the step time
    of the full workload's layer count is extrapolated by the caller."""
    from oracle import oracle as ora
    code = ora.dtype_code(w.dtype)
    reqs = list(range(m))
    q, Ks, Vs = _host_batch(w, reqs)
    ks, vs = wl.e4m3_scales(1)
    store = ora.KVStore(1, w.kv_heads, w.head_dim, code, kv_e4m3=w.kv_dtype == "e4m3", k_scale=ks, v_scale=vs)
    for r, k, v in zip(reqs, Ks, Vs):
        store.append(r, 0, k[:-1], v[:-1])
        store.gathered(r, 0)
    t0 = time.perf_counter()
    for r, k, v in zip(reqs, Ks, Vs):                      # the step's append ...
        store.append(r, 0, k[-1:], v[-1:])
    _, _, threads = store.decode_attention(0, reqs, q, w.q_heads)     # ... and attention
    dt = time.perf_counter() - t0
    return dt, threads


def run_reference(args):
    """`--impl reference`: the CPU checker as it stands, on the host cores, same metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total = args.steps + args.warmup
    w, step_layers, copies = pick_workload(args.workload, kv_dtype=args.kv_dtype)
    per_step_budget = max(0.02, min(15.0, 150.0 / max(total, 1)))
    m, _ = checker_sample(w, step_layers, per_step_budget)
    times, threads = [], 0
    for i in range(total):
        dt, threads = checker_time_step(w, m, step_layers)
        if i >= args.warmup:
            times.append(dt)
    t_step = sum(times) / len(times) * step_layers         # all stepped layers cost the same
    value = m / t_step
    sample = (f"first {m} of {w.batch} requests ({int((w.context[:m] + 1).sum())} of "
              f"{int((w.context + 1).sum())} KV tokens), one layer timed"
              + (f", x{step_layers} layers" if step_layers > 1 else ""))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args.workload, step_layers, copies),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# the GPU arm
# ---------------------------------------------------------------------------------------------

def workload_config(w, name, step_layers, copies):
    desc = {"config2": "configs[1]: Qwen-7B-shaped single layer, 28q/4kv heads, head_dim 128, bf16, batch 64, "
                       "contexts lognormal(median 512, sigma 0.8) in [16,8192], quartile buckets",
            "config3": "configs[2]: 28-layer Qwen-7B-shaped pool of 40 GB, batch 256, Pareto(1.5, 32) lengths, "
                       "noisy predictions, 10% safety pool",
            "config5": "configs[4]: long-reasoning decode, batch 32, contexts U[16384,32768], 28 layers"}[name]
    kv_bytes_layer = int((w.context + 1).sum()) * 2 * w.kv_heads * w.head_dim * w.elem_bytes
    if w.kv_dtype == "e4m3":
        desc += "; K/V slabs held as E4M3 codes with per-layer scales (q, new rows and output bf16)"
    return {"workload": desc, "batch": w.batch, "layers_per_step": step_layers,
            "kv_tokens": int((w.context + 1).sum()), "kv_bytes_per_layer": kv_bytes_layer,
            "l2": (f"steps rotate over {copies} independent KV copies ({copies * kv_bytes_layer >> 20} MiB > L2)"
                   if copies > 1 else f"one step streams {step_layers * kv_bytes_layer >> 20} MiB of KV (> L2)"),
            "overlap": "consecutive launches are on different layers (KV copies) of one pool and do not wait for one "
                       "another, as the layers of a model do not; roofline.serialised has the same steps with every "
                       "launch waiting for the one before"}


def kernel_sources_hash() -> str:
    """sha256 over the CUDA/C++ sources of the library: identifies the kernels a counter capture
    was taken from."""
    import glob
    import hashlib
    h = hashlib.sha256()
    base = os.path.join(ROOT, "paper_2512_09427_b200", "csrc")
    for f in sorted(glob.glob(os.path.join(base, "*"))):
        h.update(os.path.basename(f).encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, kernel: str):
    """DRAM bytes (read + written) per launch of the decode kernel from the ncu capture noted in
    profiles/traffic.json, or None when there is no capture of this kernel on this workload or
    the kernel sources have changed since it was taken."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f)[f"{workload}:{kernel}"]
    except Exception:
        return None
    if rec.get("sources_sha256_16") != kernel_sources_hash():
        return None
    return float(rec["dram_bytes_per_launch"])


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def run_ours(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    phases = set(args.phases.split(","))
    K, W = args.steps, args.warmup
    w, step_layers, copies = pick_workload(args.workload, rank, args.copies, args.layers, args.kv_dtype)
    if w.kv_dtype == "e4m3":
        phases -= {"probe", "paged"}          # both exist for 16-bit slabs only
    sd = SlabDecode(w, step_layers, dev, fused=args.fused_combine, decode_kernel=DECODE_KERNELS[args.decode_kernel])
    bounds, epoch = sd.learn_boundaries()
    sd.admit_and_fill()
    q, kn, vn, out = sd.make_inputs()
    torch.cuda.synchronize()

    odma = sd.odma
    tables = odma.Tables()
    clocks = ClockSampler(local) if "clocks" in phases else None
    peak, peak_kind = measured_peak()
    row_bytes = w.head_dim * w.elem_bytes             # of a stored K/V row
    io_row_bytes = w.head_dim * (4 if w.dtype == torch.float32 else 2)
    n = w.batch
    step_no = 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- warm-up, then regions of exactly K timed steps ------------------------------------------
    # One region = m x K consecutive steps (m = 1 for K >= 256) between two CUDA events on the launch stream.  A region of
    # the default K lasts a fraction of a millisecond, so regions are enqueued back to back until
    # MIN_TIMED_SECONDS of device time have been timed (no host synchronisation in between);
    # `ms_per_step` is the median region, the spread is reported beside it.  Barrier and
    # synchronize bracket the whole timed part, and the clock sampler covers exactly it.
    for _ in range(W):
        sd.step(step_no, q, kn, vn, out, tables)
        step_no += 1
    # what one step launches (a step over several layers may be ONE decode launch)
    sd.pool.profile_enable(True)
    sd.step(step_no, q, kn, vn, out, tables)
    step_no += 1
    torch.cuda.synchronize()
    dec_per_step = sd.pool.profile_read(odma.K_DECODE)[1]
    other_per_step = sd.pool.profile_read(odma.K_APPEND)[1] + sd.pool.profile_read(odma.K_COMBINE)[1]
    sd.pool.profile_enable(False)
    barrier()
    ev0.record()
    for _ in range(max(W, 3)):
        sd.step(step_no, q, kn, vn, out, tables)
        step_no += 1
    ev1.record()
    torch.cuda.synchronize()
    est_ms = max_over_ranks([ev0.elapsed_time(ev1) / max(W, 3)], dist, dev)[0]
    KR = K * max(1, -(-MIN_REGION_STEPS // K))        # steps per timed region: m x K
    n_regions = int(min(5000, max(5, -(-MIN_TIMED_SECONDS * 1e3 // max(KR * est_ms, 1e-6)))))
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_regions + 1)]
    barrier()
    t_wall0 = time.time()
    marks[0].record()
    for r in range(n_regions):
        for _ in range(KR):
            sd.step(step_no, q, kn, vn, out, tables)
            step_no += 1
        marks[r + 1].record()
    barrier()
    if clocks:
        clocks.mark(t_wall0, time.time())
    region_ms = max_over_ranks([marks[r].elapsed_time(marks[r + 1]) for r in range(n_regions)], dist, dev)
    region_ms = [x * K / KR for x in region_ms]       # per K steps
    ms = statistics.median(region_ms)
    assert sd.pool.check_status(sd.stream) == odma.OK
    launches_per_step = dec_per_step + other_per_step
    kv_bytes_layer = tables.kv_tokens * 2 * w.kv_heads * row_bytes
    kv_bytes_per_launch = kv_bytes_layer * step_layers // dec_per_step     # a launch may cover all layers of the step
    step_bytes = step_layers * (kv_bytes_layer + 2 * n * w.q_heads * io_row_bytes + 2 * n * w.kv_heads * io_row_bytes)
    if w.dtype != torch.bfloat16:
        kernel_name = "decode_generic_kernel"
    elif args.decode_kernel in ("tcgen05", "auto") or w.kv_dtype == "e4m3":
        # auto: every step but the very first follows a decode step on another layer (another KV copy)
        # and runs on the tcgen05 kernel, chained; the mma.sync kernel serves launches that have to wait
        kernel_name = "decode_umma_kernel"
    else:
        kernel_name = "decode_tc_kernel"

    # ---- the same steps with every launch bracketed by CUDA events (per-kernel time) ----------
    roofline, kernels_us = None, None
    if "kernels" in phases:
        prof_steps = max(3, min(K, 500))
        sd.pool.profile_enable(True)
        t0w = time.time()
        for _ in range(prof_steps):
            sd.step(step_no, q, kn, vn, out, tables)
            step_no += 1
        torch.cuda.synchronize()
        if clocks:
            clocks.mark(t0w, time.time())
        dec_ms, dec_n = sd.pool.profile_read(odma.K_DECODE)
        app_ms, app_n = sd.pool.profile_read(odma.K_APPEND)
        cmb_ms, cmb_n = sd.pool.profile_read(odma.K_COMBINE)
        sd.pool.profile_enable(False)
        # The decode kernel's launch duration.  When a step is nothing but that kernel (append and
        # merge fused into it) the timed region above IS a run of K x layers launches between two
        # CUDA events on the launch stream: its average is the figure.  Otherwise the launches
        # bracketed one by one are used (each bracket adds the events' own latency).
        bracketed_us = dec_ms / dec_n * 1e3
        if other_per_step == 0:
            us, how, timed_n = (ms / (K * dec_per_step) * 1e3, f"median timed region: {KR} steps of consecutive launches between two events",
                                KR * dec_per_step)
        else:
            us, how, timed_n = bracketed_us, "each launch bracketed by two events", dec_n
        achieved = kv_bytes_per_launch / (us * 1e-6) / 1e9
        isolated = kv_bytes_per_launch / (bracketed_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                    "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                    "traffic": recorded_traffic(args.workload + ("-e4m3" if w.kv_dtype == "e4m3" else ""), kernel_name),
                    "bytes_per_launch": kv_bytes_per_launch, "us_per_launch": us, "timing": how,
                    "launches_timed": timed_n, "us_per_launch_bracketed": bracketed_us,
                    "frac_isolated": isolated / peak, "layers_per_launch": step_layers // dec_per_step}
        kernels_us = {"append": app_ms / max(app_n, 1) * 1e3, "decode": dec_ms / dec_n * 1e3,
                      "combine": cmb_ms / cmb_n * 1e3 if cmb_n else 0.0}

    # ---- the same steps with every launch made to wait for the one before (chain_launches = 0) ----
    # A second pool over the same, already filled memory (same slabs: the allocator is deterministic).
    if "serial" in phases and roofline is not None:
        sd0 = SlabDecode(w, step_layers, dev, fused=args.fused_combine, decode_kernel=DECODE_KERNELS[args.decode_kernel],
                         chain_launches=0, mem=sd.mem)
        sd0.learn_boundaries()
        sd0.admit_and_fill(fill=False)
        t0 = odma.Tables()
        i0 = 0
        for _ in range(max(W, 3)):
            sd0.step(i0, q, kn, vn, out, t0)
            i0 += 1
        torch.cuda.synchronize()
        reps = max(5, min(n_regions, 50))
        sm = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        t0w = time.time()
        sm[0].record()
        for r in range(reps):
            for _ in range(K):
                sd0.step(i0, q, kn, vn, out, t0)
                i0 += 1
            sm[r + 1].record()
        torch.cuda.synchronize()
        if clocks:
            clocks.mark(t0w, time.time())
        assert sd0.pool.check_status(sd0.stream) == odma.OK
        s_us = statistics.median(sm[r].elapsed_time(sm[r + 1]) for r in range(reps)) / (K * dec_per_step) * 1e3
        roofline["serialised"] = {"us_per_launch": s_us, "frac": kv_bytes_per_launch / (s_us * 1e-6) / 1e9 / peak,
                                  "what": "the same steps with chain_launches = 0: every launch waits for the kernel ahead of it"}
        sd0.pool.destroy()

    # ---- the read probe: the decode kernel's loads and barrier traffic with no arithmetic, launched
    #      the way the timed steps are (consecutive launches between two events)
    probe_line = None
    if "probe" in phases and w.dtype == torch.bfloat16:
        own_p = torch.empty(sd.pool.tables_bytes(n), dtype=torch.uint8, device=dev)
        tables_p = sd.pool.build_tables(sd.reqs, own_p.data_ptr(), own_p.numel(), sd.stream)
        reps = max(20, min(K, 200)) if step_layers == 1 else 2
        for timed in (False, True):
            if timed:
                ev0.record()
            for i in range(reps * step_layers):
                sd.pool.read_probe(i % w.layers, w.q_heads, tables_p, sd.stream)
            if timed:
                ev1.record()
            torch.cuda.synchronize()
        assert sd.pool.check_status(sd.stream) == odma.OK
        p_us = ev0.elapsed_time(ev1) / (reps * step_layers) * 1e3
        probe_line = {"us_per_launch": p_us, "GBs": kv_bytes_layer / (p_us * 1e-6) / 1e9,
                      "frac": kv_bytes_layer / (p_us * 1e-6) / 1e9 / peak, "launches": reps * step_layers,
                      "kernel": "decode_tc_kernel<probe>"}
        del own_p

    # ---- contiguity ablation: the same requests re-laid in 16-token pages (shuffled), same kernel
    paged_line = None
    if "paged" in phases:
        host_len = [int(c) + 1 for c in w.context]
        max_pages = max(-(-L // 16) for L in host_len)
        n_pages = sum(-(-L // 16) for L in host_len) + 16
        page_bytes = w.layers * 2 * w.kv_heads * 16 * row_bytes
        pages = torch.empty(n_pages * page_bytes, dtype=torch.uint8, device=dev)
        ptab = torch.zeros(n * max_pages, dtype=torch.int32, device=dev)
        paged = odma.Paged(sd.pool, pages.data_ptr(), pages.numel())
        own = torch.empty(sd.pool.tables_bytes(n), dtype=torch.uint8, device=dev)
        # tables of the ablation's own: context+1 tokens, the last one written by the steps above
        tables_a = sd.pool.build_tables(sd.reqs, own.data_ptr(), own.numel(), sd.stream)
        paged.build(tables_a, host_len, 950900, ptab.data_ptr(), max_pages, sd.stream)
        reps = max(3, min(K, 200)) if step_layers == 1 else 3
        res = {}
        for kind in ("slab", "paged"):
            for timed in (False, True):
                if timed:
                    sd.pool.profile_enable(True)
                for i in range(reps * step_layers):
                    l = i % w.layers
                    if kind == "slab":
                        sd.pool.decode_attention(l, q[l].data_ptr(), w.q_heads, tables_a, out[l].data_ptr(), 0, sd.stream)
                    else:
                        paged.decode_attention(l, q[l].data_ptr(), w.q_heads, tables_a, ptab.data_ptr(), max_pages,
                                               out[l].data_ptr(), 0, sd.stream)
                torch.cuda.synchronize()
            t_ms, cnt = sd.pool.profile_read(odma.K_DECODE)
            sd.pool.profile_enable(False)
            res[kind] = {"us_per_launch": t_ms / cnt * 1e3, "GBs": kv_bytes_layer / (t_ms / cnt * 1e-3) / 1e9}
        assert sd.pool.check_status(sd.stream) == odma.OK
        paged_line = {"pages": "16 tokens, ids shuffled", "timing": "each launch bracketed by two events", **res,
                      "slab_over_paged": res["paged"]["us_per_launch"] / res["slab"]["us_per_launch"]}
        del pages, paged

    # ---- end to end from pinned host buffers ---------------------------------------------------
    e2e = None
    if "e2e" in phases:
        e2e_steps = max(3, min(K, 200))
        hq, hkn, hvn, hout = sd.make_inputs(pinned=True)
        for _ in range(3):
            sd.step_host(step_no, hq, hkn, hvn, hout)
            step_no += 1
        barrier()
        t0w = time.time()
        ev0.record()
        for _ in range(e2e_steps):
            sd.step_host(step_no, hq, hkn, hvn, hout)
            step_no += 1
        ev1.record()
        barrier()
        if clocks:
            clocks.mark(t0w, time.time())
        e2e_ms = ev0.elapsed_time(ev1)
        assert sd.pool.check_status(sd.stream) == odma.OK
    else:
        e2e_steps, e2e_ms = 1, float("nan")

    clk = clocks.stop() if clocks else None

    # ---- max over ranks ------------------------------------------------------------------------
    e2e_ms = max_over_ranks([e2e_ms], dist, dev)[0]
    value = world * n * K / (ms * 1e-3)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "e4m3" if w.kv_dtype == "e4m3" else "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
            "config": workload_config(w, args.workload, step_layers, copies),
            "regions": {"count": n_regions, "steps_each": KR, "ms_per_step_min": min(region_ms) / K,
                        "ms_per_step_max": max(region_ms) / K, "timed_seconds": sum(region_ms) * KR / K * 1e-3},
            "step_gbs": step_bytes / (ms / K * 1e-3) / 1e9,
            "gpu_launches": int(launches_per_step * K),
            "plan": {"ctas": tables.n_ctas, "items": tables.n_items, "combine": tables.n_combine},
            "buckets": list(bounds), "migrations_at_fill": sd.migrations_at_fill}
    if e2e_ms == e2e_ms:
        h2d = step_layers * (n * w.q_heads * io_row_bytes + 2 * n * w.kv_heads * io_row_bytes + tables.words * 4)
        d2h = step_layers * n * w.q_heads * io_row_bytes
        line["e2e"] = {"value": world * n * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                       "ms_per_step": e2e_ms / e2e_steps}
    if roofline:
        line["roofline"], line["kernels_us"] = roofline, kernels_us
    if probe_line:
        line["read_probe"] = probe_line
        line["read_probe_gbs"] = probe_line["GBs"]
    if paged_line:
        line["page16_ablation"] = paged_line
    if clk:
        line["clocks"] = clk
    if rank == 0 and world == 1 and "cpu" in phases:
        m, _ = checker_sample(w, step_layers, 4.0)
        dts = []
        threads = 0
        for _ in range(3):
            dt, threads = checker_time_step(w, m, step_layers)
            dts.append(dt)
        t_step = min(dts) * step_layers
        line["cpu_baseline"] = {"value": m / t_step, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"first {m} of {w.batch} requests, one layer, best of 3"
                                          + (f", x{step_layers} layers" if step_layers > 1 else "")}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_config4(args):
    """`--workload config4`: the drift stream through the allocator on the host (utilisation,
    migrations, boundaries), then the decode step of the live batch of each half on the GPU."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    stats, halves = config4_drift()
    peak, peak_kind = measured_peak()
    K, W = args.steps, args.warmup
    out_halves = []
    for name, epoch, w in halves:
        kv_bytes = int((w.context + 1).sum()) * 2 * w.kv_heads * w.head_dim * w.elem_bytes
        copies = max(2, -(-3 * L2_BYTES // kv_bytes))               # rotate over copies: cold L2
        wc = wl.scaled(w, layers=copies, pool_bytes=w.pool_bytes * copies)
        sd = SlabDecode(wc, 1, dev, fused=args.fused_combine, decode_kernel=DECODE_KERNELS[args.decode_kernel])
        sd.learn_boundaries()
        sd.admit_and_fill()
        q, kn, vn, out = sd.make_inputs()
        tables = sd.odma.Tables()
        for i in range(W):
            sd.step(i, q, kn, vn, out, tables)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for i in range(K):
            sd.step(W + i, q, kn, vn, out, tables)
        ev1.record()
        torch.cuda.synchronize()
        assert sd.pool.check_status(sd.stream) == sd.odma.OK
        ms = ev0.elapsed_time(ev1) / K
        st = sd.pool.get_stats()
        out_halves.append({"half": name, "epoch": epoch, "batch": wc.batch, "kv_tokens": int(tables.kv_tokens),
                           "ms_per_step": ms, "tokens_per_s": wc.batch / (ms * 1e-3),
                           "decode_gbs": kv_bytes / (ms * 1e-3) / 1e9, "frac_of_peak": kv_bytes / (ms * 1e-3) / 1e9 / peak,
                           "batch_utilisation": st["used_live"] / max(st["reserved_live"], 1),
                           "plan": {"ctas": tables.n_ctas, "items": tables.n_items, "combine": tables.n_combine},
                           "kv_copies": copies})
        del sd, q, kn, vn, out
        torch.cuda.empty_cache()
    line = {"metric": METRIC, "value": out_halves[0]["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": out_halves[0]["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "configs[3]: drift stream, 10,000 requests, rebucketing every 500, 28q/4kv/128 bf16 single "
                                   "layer, steady-state batch 128; `value` is the first half's batch, both halves below"},
            "allocator": stats, "halves": out_halves, "peak": peak, "peak_kind": peak_kind}
    print(json.dumps(line), flush=True)


def run_prefill(args):
    """`--workload prefill`: a chunk of prompt tokens per request appended to Qwen-7B-shaped slabs and
    attended causally (odma_build_prefill_tables + the decode kernel: one stream per new token).  The
    timed step is the chunk's attention on one layer; copies of the layer rotate so that L2 starts cold."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    from paper_2512_09427_b200 import odma
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    K, W = args.steps, args.warmup
    n_req, ctx, chunk, copies = 8, 1920, 128, 8
    context = np.full(n_req, ctx, dtype=np.int64)
    w = wl.Workload(name="prefill", seed=950907, layers=copies, q_heads=28, kv_heads=4, head_dim=128, dtype=torch.bfloat16,
                    pool_bytes=copies * n_req * 4096 * 2 * 4 * 128 * 2 * 2, safety_pct=10, max_len=4096, context=context,
                    predicted=context + chunk, static_buckets=(2048, 4096))
    if args.kv_dtype == "e4m3":
        w = wl.with_e4m3(w)
    sd = SlabDecode(w, 1, dev, fused=args.fused_combine, decode_kernel=DECODE_KERNELS[args.decode_kernel])
    sd.learn_boundaries()
    sd.admit_and_fill()
    pool, reqs = sd.pool, sd.reqs
    # the chunk: appended on every layer copy through the ordinary calls, its plan made first
    for r in reqs:
        rc, _, _ = pool.ensure_capacity(r, ctx + chunk, sd.stream)
        assert rc == odma.OK
    table = torch.empty(pool.tables_bytes(n_req * chunk), dtype=torch.uint8, device=dev)
    pt = pool.build_prefill_tables(reqs, [chunk] * n_req, table.data_ptr(), table.numel(), sd.stream)
    table_app = torch.empty(pool.tables_bytes(n_req), dtype=torch.uint8, device=dev)
    t_app = pool.build_tables(reqs, table_app.data_ptr(), table_app.numel(), sd.stream, [chunk] * n_req)
    for layer in range(copies):
        kk = torch.cat([wl.kv_rows(w.seed, layer, r, wl.KIND_K, ctx, ctx + chunk, 4, 128, w.dtype, dev) for r in reqs])
        vv = torch.cat([wl.kv_rows(w.seed, layer, r, wl.KIND_V, ctx, ctx + chunk, 4, 128, w.dtype, dev) for r in reqs])
        pool.append_kv(layer, t_app, kk.data_ptr(), vv.data_ptr(), sd.stream)
        torch.cuda.synchronize()
    q = torch.stack([torch.cat([torch.stack([wl.q_rows(w.seed, layer, r, j, 28, 128, w.dtype, dev) for j in range(chunk)])
                                for r in reqs]) for layer in range(copies)]).contiguous()
    out = torch.zeros_like(q)
    def step(i):
        l = i % copies
        pool.decode_attention(l, q[l].data_ptr(), 28, pt, out[l].data_ptr(), 0, sd.stream)
    for i in range(max(W, 3)):
        step(i)
    torch.cuda.synchronize()
    clocks = ClockSampler(dev.index or 0)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
    t0 = time.time()
    ev[0].record()
    for r in range(5):
        for i in range(K):
            step(r * K + i)
        ev[r + 1].record()
    torch.cuda.synchronize()
    clocks.mark(t0, time.time())
    assert pool.check_status(sd.stream) == odma.OK
    ms = statistics.median(ev[r].elapsed_time(ev[r + 1]) for r in range(5)) / K
    keys = sum(ctx + j + 1 for j in range(chunk)) * n_req                 # (token, key) pairs per KV head
    flops = 2 * 2 * keys * 28 * 128                                      # two products, 28 query heads
    read_once = n_req * (ctx + chunk) * 2 * 4 * 128 * w.elem_bytes       # the slabs read once
    read_per_token = keys * 2 * 4 * 128 * w.elem_bytes                   # what this form reads (per new token, from L2 after the first)
    line = {"metric": "prefill tokens/s (chunk attention over the slabs, one layer)", "value": n_req * chunk / (ms * 1e-3),
            "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3" if w.kv_dtype == "e4m3" else "bf16", "data": "synthetic",
            "config": {"workload": f"chunked prefill: {n_req} requests, context {ctx}, chunk {chunk} tokens, Qwen-7B-shaped layer "
                                   f"(28q/4kv heads, head_dim 128), {copies} rotating layer copies",
                       "streams": int(pt.n), "items": int(pt.n_items), "split_streams": int(pt.n_combine)},
            "gpu_launches": K,
            "roofline": {"bound": "hbm", "kernel": "decode_tc_kernel" if args.decode_kernel != "tcgen05" and w.kv_dtype != "e4m3" else "decode_umma_kernel",
                         "achieved": read_per_token / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                         "frac": read_per_token / (ms * 1e-3) / 1e9 / peak, "peak_kind": peak_kind, "traffic": None,
                         "bytes_per_launch": read_per_token, "us_per_launch": ms * 1e3,
                         "note": "bytes = the slab prefix of every new token (this form streams it once per token, mostly from L2); "
                                 "the slabs themselves are " + str(read_once) + " bytes; tensor work " + str(flops) + " flop"},
            "tflops": flops / (ms * 1e-3) / 1e12, "clocks": clocks.stop()}
    print(json.dumps(line), flush=True)


def run_admission(args):
    """`--workload admission`: the paper's serving protocol (Section V) on the library's native
    simulator.  Two decode launches of the config-2 shape (full batch and half of it) are timed
    on the GPU and fitted to  t = base + per_token * kv_tokens ; with that step-time model a
    Poisson request trace is run through one 28-layer replica over a 40 GB pool under static
    worst-case reservation, 16-token pages and the ODMA allocator (with and without the
    predictor's uncertainty).  Reports utilisation, admitted concurrency and tokens/s."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the step-time model is measured, not assumed")
    from paper_2512_09427_b200 import odma
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    points = []
    for frac in (1.0, 0.5):
        w, step_layers, copies = pick_workload("config2", 0, args.copies)
        if frac < 1.0:
            m = int(w.batch * frac)
            w = wl.scaled(w, context=w.context[:m], predicted=w.predicted[:m])
        sd = SlabDecode(w, 1, dev, fused=args.fused_combine, decode_kernel=DECODE_KERNELS[args.decode_kernel])
        sd.learn_boundaries()
        sd.admit_and_fill()
        q, kn, vn, out = sd.make_inputs()
        tables = odma.Tables()
        for i in range(20):
            sd.step(i, q, kn, vn, out, tables)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(200, args.steps)
        ev0.record()
        for i in range(reps):
            sd.step(20 + i, q, kn, vn, out, tables)
        ev1.record()
        torch.cuda.synchronize()
        points.append((int(tables.kv_tokens), ev0.elapsed_time(ev1) / reps * 1e6))     # (tokens, ns per launch)
        del sd, q, kn, vn, out
        torch.cuda.empty_cache()
    (t1, n1), (t2, n2) = points
    per_token_ns = (n1 - n2) / (t1 - t2)
    base_ns = max(0.0, n1 - per_token_ns * t1)
    ps_per_token = int(round(per_token_ns * 1000))
    layers, max_len, max_batch = 28, 8192 + 16, 256
    pool_bytes = 40 * 10**9
    n_req = args.requests
    results = {}
    # offered load: what the static policy can just not keep up with (its concurrency is pool / max_len)
    token_bytes = layers * 2 * 4 * 128 * 2
    static_conc = pool_bytes // token_bytes // max_len
    mean_total = 700.0                                             # lognormal(512, 0.8) clipped: mean about 700 tokens
    step_s = layers * (base_ns + ps_per_token * 1e-3 * static_conc * mean_total * 0.6) * 1e-9
    rate = args.rate or 1.5 * static_conc / (mean_total * 0.75 * step_s)
    for name, policy, unc in (("static", odma.SIM_STATIC, False), ("page16", odma.SIM_PAGED16, False),
                              ("odma", odma.SIM_ODMA, False), ("odma_uncertainty", odma.SIM_ODMA, True)):
        rows = wl.poisson_trace(950906, n_req, rate, law="lognormal", max_len=max_len - 16, with_uncertainty=unc)
        cfg = odma.config_default()
        cfg.safety_pct, cfg.max_len, cfg.window, cfg.refresh = 10, max_len, 2000, 500
        pool = odma.Pool(0, pool_bytes, layers, 4, 128, odma.DTYPE_BF16, cfg)
        assert pool.set_buckets([304, 528, 912, 8192]) == 0        # the quartile boundaries config 2 learns
        t0 = time.perf_counter()
        r = pool.sim_run(policy, rows, max_batch, layers, int(round(base_ns)), ps_per_token)
        r["host_seconds"] = time.perf_counter() - t0
        r["utilisation"] = r["sum_actual"] / max(r["sum_reserved"], 1)
        r["utilisation_time_avg"] = r["used_time"] / max(r["reserved_time"], 1)
        r["mean_concurrency"] = r["conc_time"] / max(r["makespan_ns"], 1)
        r["tokens_per_s"] = r["tokens_out"] / max(r["makespan_ns"], 1) * 1e9
        results[name] = r
    base = results["static"]
    line = {"metric": "admission simulation: KV utilisation, admitted concurrency and decode tokens/s under three reservation policies",
            "value": results["odma"]["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": None, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": "Poisson arrivals (lognormal(512, 0.8) totals, prompt = total/4, prediction error "
                                   "lognormal(0, 0.3)) into a 40 GB, 28-layer Qwen-7B-shaped pool, max_batch 256",
                       "requests": n_req, "arrival_rate_per_s": rate, "max_len": max_len},
            "step_time_model": {"base_ns_per_layer": base_ns, "ps_per_kv_token_per_layer": ps_per_token,
                                "fitted_from": [{"kv_tokens": t, "ns_per_launch": n} for t, n in points]},
            "policies": results,
            "odma_vs_static": {"utilisation_gain_abs": results["odma"]["utilisation"] - base["utilisation"],
                               "tokens_per_s_ratio": results["odma"]["tokens_per_s"] / max(base["tokens_per_s"], 1e-9),
                               "concurrency_ratio": results["odma"]["mean_concurrency"] / max(base["mean_concurrency"], 1e-9)},
            "paper_context": "the paper reports up to +19.25 % absolute KV utilisation and +23-27 % tokens/s over static "
                             "reservation on Cambricon MLU370-X4 with Alpaca / Google-NQ (its Section V); other hardware, "
                             "other data: context, not a target"}
    print(json.dumps(line), flush=True)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    t = torch.nan_to_num(t, nan=-1.0)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) if v >= 0 else float("nan") for v in t]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="config2", choices=["config2", "config3", "config4", "config5", "admission", "prefill"])
    ap.add_argument("--requests", type=int, default=4000, help="admission: requests in the Poisson trace")
    ap.add_argument("--rate", type=float, default=0.0, help="admission: arrivals per second (0 = 1.5x what static reservation sustains)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--phases", default="",
                    help="comma list of the passes to run besides the timed one: kernels (per-kernel CUDA-event "
                         "times), serial (the steps again with every launch waiting for the one before), e2e (host buffers), "
                         "clocks (nvidia-smi sampler), cpu (CPU checker baseline), "
                         "probe (the no-arithmetic read probe), paged (page-16 ablation of the decode kernel on "
                         "the same inputs); default: all of them on config2, all but paged elsewhere")
    ap.add_argument("--fused-combine", type=int, default=1, help="1: split streams merged inside the decode kernel")
    ap.add_argument("--decode-kernel", default="auto", choices=list(DECODE_KERNELS),
                    help="which bf16 decode kernel the pool runs (auto: the library's choice per shape)")
    ap.add_argument("--readout", default="auto", choices=["auto", "late", "at_once"],
                    help="tcgen05 kernel, 16-bit slabs: when an item's result is read out of tensor memory (auto: per launch, by the plan's counts)")
    ap.add_argument("--kv-dtype", default="bf16", choices=["bf16", "e4m3"],
                    help="element type of the slabs: bf16 (the configs as stated) or E4M3 codes with per-layer scales")
    ap.add_argument("--copies", type=int, default=0, help="config2: rotating KV copies (0 = enough for 3x L2)")
    ap.add_argument("--layers", type=int, default=0,
                    help="config3/config5: step through this many layers only (0 = all 28; a reduced size for profiler "
                         "captures, not the benchmark configuration)")
    args = ap.parse_args()
    global READOUT
    READOUT = {"auto": 0, "late": 1, "at_once": 2}[args.readout]
    if args.warmup < 3:
        args.warmup = 3
    if not args.phases:
        args.phases = "timed,kernels,serial,e2e,clocks,cpu,probe" + (",paged" if args.workload == "config2" else "")
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "config4":
        run_config4(args)
    elif args.workload == "prefill":
        run_prefill(args)
    elif args.workload == "admission":
        run_admission(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
