"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

This module holds no arithmetic of the method itself (no attention, no
allocation policy).  It only produces inputs:

* request-length traces with the shapes of the five evaluation workloads
  (log-normal, Pareto, drifting bimodal, uniform long-context),
* Q/K/V values ~N(0,1) from a counter-based generator, so that any element of
  any tensor can be regenerated on the CPU or on the GPU, bit for bit, without
  ever storing the tensor (needed for the 40-60 GB pools),
* a small closed-loop serving driver (fixed concurrency, one token per step)
  that turns a length trace into the alloc / grow / free event sequence an
  allocator sees.

They stand in for the Alpaca / Google-NQ request streams and the
DeepSeek-R1-Distill-Qwen-7B activations of the paper's evaluation (Section V),
none of which are available offline.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

_M32 = 0xFFFFFFFF
_TABLE_BITS = 16

# ---------------------------------------------------------------------------
# counter-based N(0,1) generator (integer hash -> quantile table lookup)
# ---------------------------------------------------------------------------


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for 0 <= x < 2^32 held in int64, without int64 overflow."""
    hi = ((x >> 16) * c) & 0xFFFF
    lo = (x & 0xFFFF) * c
    return ((hi << 16) + lo) & _M32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """A 32-bit integer finaliser (xor-shift / multiply rounds) on int64 tensors."""
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def fold_key(key: Sequence[int]) -> int:
    """Fold a tuple of non-negative ints into one 32-bit stream seed."""
    s = 0x9E3779B9
    for k in key:
        k = int(k)
        s = _mix32_int(s ^ (k & _M32))
        s = _mix32_int(s ^ ((k >> 32) & _M32) ^ 0x85EBCA6B)
    return s


_tables: Dict[Tuple[str, str], torch.Tensor] = {}


def _normal_table(dtype: torch.dtype, device: torch.device) -> torch.Tensor:
    """65536 N(0,1) quantiles, rounded to `dtype` on the CPU, then moved to `device`."""
    k = (str(dtype), str(device))
    t = _tables.get(k)
    if t is None:
        base = _tables.get((str(dtype), "cpu"))
        if base is None:
            n = 1 << _TABLE_BITS
            p = (torch.arange(n, dtype=torch.float64) + 0.5) / n
            base = torch.special.ndtri(p).to(torch.float32).to(dtype)
            _tables[(str(dtype), "cpu")] = base
        t = base.to(device)
        _tables[k] = t
    return t


def gen_normal(key: Sequence[int], start: int, count: int, dtype: torch.dtype,
               device="cpu") -> torch.Tensor:
    """Elements [start, start+count) of the N(0,1) stream named by `key`, in `dtype`.

    Pure integer hashing followed by a table lookup, so CPU and CUDA give the
    same bits for the same (key, index).
    """
    device = torch.device(device)
    s = fold_key(key)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    lo = idx & _M32
    hi = idx >> 32
    h = _mix32(lo ^ _mix32(hi ^ s))
    return _normal_table(dtype, device)[h & ((1 << _TABLE_BITS) - 1)]


KIND_Q, KIND_K, KIND_V = 0, 1, 2


def kv_rows(seed: int, layer: int, req: int, kind: int, t0: int, t1: int,
            kv_heads: int, head_dim: int, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """K (kind=1) or V (kind=2) rows of tokens [t0, t1) of one request: [t1-t0, kv_heads, head_dim]."""
    per_tok = kv_heads * head_dim
    x = gen_normal((seed, layer, req, kind), t0 * per_tok, (t1 - t0) * per_tok, dtype, device)
    return x.view(t1 - t0, kv_heads, head_dim)


def kv_rows_batch(seed: int, layer: int, reqs: Sequence[int], kind: int, t0: Sequence[int],
                  t1: Sequence[int], kv_heads: int, head_dim: int, dtype: torch.dtype,
                  device="cpu") -> torch.Tensor:
    """kv_rows of several requests at once, concatenated in request order:
    [sum(t1 - t0), kv_heads, head_dim].  Element for element equal to calling kv_rows per
    request; one pass of the hash over all of them (many short runs cost one launch each
    otherwise)."""
    device = torch.device(device)
    per_tok = kv_heads * head_dim
    counts = [(int(b) - int(a)) * per_tok for a, b in zip(t0, t1)]
    total = sum(counts)
    if total == 0:
        return torch.empty(0, kv_heads, head_dim, dtype=dtype, device=device)
    seeds = torch.tensor([fold_key((seed, layer, int(r), kind)) for r in reqs], dtype=torch.int64)
    cnt = torch.tensor(counts, dtype=torch.int64)
    first = torch.tensor([int(a) * per_tok for a in t0], dtype=torch.int64)
    run_start = torch.cumsum(cnt, 0) - cnt
    s = torch.repeat_interleave(seeds, cnt).to(device)
    idx = torch.arange(total, dtype=torch.int64, device=device) + torch.repeat_interleave(first - run_start, cnt).to(device)
    lo = idx & _M32
    hi = idx >> 32
    h = _mix32(lo ^ _mix32(hi ^ s))
    return _normal_table(dtype, device)[h & ((1 << _TABLE_BITS) - 1)].view(-1, kv_heads, head_dim)


def q_rows(seed: int, layer: int, req: int, step: int, q_heads: int, head_dim: int,
           dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """The query of one request at decode step `step`: [q_heads, head_dim]."""
    x = gen_normal((seed, layer, req, KIND_Q, step), 0, q_heads * head_dim, dtype, device)
    return x.view(q_heads, head_dim)


# ---------------------------------------------------------------------------
# length laws
# ---------------------------------------------------------------------------


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def lognormal_lengths(rng, n, median, sigma, lo, hi) -> np.ndarray:
    x = np.exp(rng.normal(math.log(median), sigma, size=n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def pareto_lengths(rng, n, alpha, xmin, hi) -> np.ndarray:
    u = rng.random(size=n)
    x = xmin / np.power(1.0 - u, 1.0 / alpha)
    return np.clip(np.rint(x), xmin, hi).astype(np.int64)


def uniform_lengths(rng, n, lo, hi) -> np.ndarray:
    return rng.integers(lo, hi + 1, size=n).astype(np.int64)


def noisy_prediction(rng, true_len: np.ndarray, sigma: float) -> np.ndarray:
    f = np.exp(rng.normal(0.0, sigma, size=true_len.shape[0]))
    return np.maximum(1, np.rint(true_len * f)).astype(np.int64)


# quantile presets: p_i = num_i / den
QUARTILES = ((1, 2, 3, 4), 4)
TAIL = ((50, 80, 95, 99), 100)


@dataclass
class Workload:
    """One evaluation workload: model shape, pool, allocator settings and request lengths.

    `context` holds the KV length of each request BEFORE the decode step; the
    step appends one token and attends over context+1 keys.
    """
    name: str
    seed: int
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    dtype: torch.dtype
    pool_bytes: int
    safety_pct: int
    max_len: int
    context: np.ndarray
    predicted: np.ndarray                     # predicted total length passed to the allocator
    static_buckets: Optional[Tuple[int, ...]] = None
    warmup_lengths: Optional[np.ndarray] = None   # realised lengths observed before admission
    quantiles: Tuple[Tuple[int, ...], int] = QUARTILES
    window: int = 10000
    refresh: int = 1000
    granule: int = 16
    extra: dict = field(default_factory=dict)
    kv_dtype: str = ""                        # "": K/V stored as `dtype`; "e4m3": one byte per element

    @property
    def batch(self) -> int:
        return int(self.context.shape[0])

    @property
    def elem_bytes(self) -> int:
        """Bytes of a stored K/V element."""
        if self.kv_dtype == "e4m3":
            return 1
        return 2 if self.dtype == torch.bfloat16 else 4

    @property
    def bytes_per_token(self) -> int:
        return self.layers * 2 * self.kv_heads * self.head_dim * self.elem_bytes


def with_e4m3(w: Workload) -> Workload:
    """The same workload on 8-bit slabs: the pool holds the same number of tokens in half the bytes."""
    assert w.dtype == torch.bfloat16
    return replace(w, name=w.name + "-e4m3", kv_dtype="e4m3", pool_bytes=w.pool_bytes // 2)


def e4m3_scales(layers: int):
    """Per-layer dequantisation scales the tests and the benchmark use with N(0,1) rows: the format's
    largest value (448) then stands for 5.6 to 7 standard deviations."""
    return [0.0125 + 0.0005 * (l % 7) for l in range(layers)], [0.015 + 0.0005 * (l % 5) for l in range(layers)]


def config1(variant: str = "a") -> Workload:
    """Tiny fp32 case: 4 requests, contexts 17/64/100/250, static buckets {64,128,256}.

    Variant "a" predicts context+1 (no migration); variant "b" predicts the bare
    context, so the append pushes request 1 from 64 to 65 tokens and out of its slab.
    """
    ctx = np.array([17, 64, 100, 250], dtype=np.int64)
    pred = ctx + 1 if variant == "a" else ctx.copy()
    hkv, d, s = 1, 64, 4
    return Workload(name=f"config1{variant}", seed=950901, layers=1, q_heads=2, kv_heads=hkv,
                    head_dim=d, dtype=torch.float32, pool_bytes=1024 * 2 * hkv * d * s,
                    safety_pct=25, max_len=512, context=ctx, predicted=pred,
                    static_buckets=(64, 128, 256))


def config2(batch: int = 64, layers: int = 1, seed: int = 950902) -> Workload:
    """Qwen-7B-shaped single layer, log-normal contexts, quartile buckets from a warm-up window."""
    rng = _rng(seed)
    warm = lognormal_lengths(rng, 10000, 512, 0.8, 16, 8192)
    ctx = lognormal_lengths(rng, batch, 512, 0.8, 16, 8192)
    hkv, d = 4, 128
    per_tok = layers * 2 * hkv * d * 2
    # room for every request at the largest bucket plus the safety pool
    tokens = int((batch * 8192 + 4096) / 0.9) + 64
    return Workload(name="config2", seed=seed, layers=layers, q_heads=28, kv_heads=hkv, head_dim=d,
                    dtype=torch.bfloat16, pool_bytes=tokens * per_tok, safety_pct=10,
                    max_len=8192 + 16, context=ctx, predicted=ctx + 1, warmup_lengths=warm)


def config3(batch: int = 256, layers: int = 28, pool_bytes: int = 40 * 10**9,
            seed: int = 950903) -> Workload:
    """Full 28-layer pool, Pareto contexts, noisy predictions, 10% safety pool."""
    rng = _rng(seed)
    warm = pareto_lengths(rng, 10000, 1.5, 32, 16384)
    true_len = pareto_lengths(rng, batch, 1.5, 32, 16384)     # length AFTER the decode step
    pred = noisy_prediction(rng, true_len, 0.3)
    return Workload(name="config3", seed=seed, layers=layers, q_heads=28, kv_heads=4, head_dim=128,
                    dtype=torch.bfloat16, pool_bytes=pool_bytes, safety_pct=10, max_len=16384,
                    context=true_len - 1, predicted=pred, warmup_lengths=warm, quantiles=TAIL)


def config4_trace(n_requests: int = 10000, seed: int = 950904) -> np.ndarray:
    """Drifting request-length stream: log-normal first half, bimodal second half."""
    rng = _rng(seed)
    half = n_requests // 2
    first = lognormal_lengths(rng, half, 256, 0.7, 16, 16384)
    n2 = n_requests - half
    is_long = rng.random(size=n2) < 0.3
    short = lognormal_lengths(rng, n2, 128, 0.7, 16, 16384)
    long_ = lognormal_lengths(rng, n2, 4096, 0.7, 16, 16384)
    second = np.where(is_long, long_, short)
    return np.concatenate([first, second]).astype(np.int64)


def config4(n_requests: int = 10000, seed: int = 950904, pool_bytes: int = 4 * 10**9,
            window: int = 2000, refresh: int = 500, noisy: bool = False,
            quantiles=QUARTILES) -> Workload:
    total = config4_trace(n_requests, seed)
    pred = noisy_prediction(_rng(seed + 7), total, 0.3) if noisy else total.copy()
    return Workload(name="config4", seed=seed, layers=1, q_heads=28, kv_heads=4, head_dim=128,
                    dtype=torch.bfloat16, pool_bytes=pool_bytes, safety_pct=10, max_len=16384,
                    context=total, predicted=pred, static_buckets=(256, 512, 1024, 16384),
                    quantiles=quantiles, window=window, refresh=refresh,
                    extra={"concurrency": 128})


def config5(batch: int = 32, layers: int = 28, pool_bytes: int = 64 * 10**9,
            lo: int = 16384, hi: int = 32768, seed: int = 950905) -> Workload:
    """Long-reasoning decode: uniform long contexts, quartile buckets of the same law."""
    rng = _rng(seed)
    warm = uniform_lengths(rng, 10000, lo, hi) + 1
    ctx = uniform_lengths(rng, batch, lo, hi)
    return Workload(name="config5", seed=seed, layers=layers, q_heads=28, kv_heads=4, head_dim=128,
                    dtype=torch.bfloat16, pool_bytes=pool_bytes, safety_pct=10,
                    max_len=hi + 4096, context=ctx, predicted=ctx + 1, warmup_lengths=warm)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of `w` with some fields replaced (used for reduced-size parity cases)."""
    d = dict(w.__dict__)
    d.update(kw)
    return Workload(**d)


# ---------------------------------------------------------------------------
# closed-loop serving driver (fixed concurrency, one token per request per step)
# ---------------------------------------------------------------------------


@dataclass
class DriftResult:
    events: int = 0
    steps: int = 0
    migrations: int = 0
    admitted: int = 0
    deferred: int = 0
    preempted: int = 0
    boundary_log: List[Tuple[int, Tuple[int, ...]]] = field(default_factory=list)


def run_closed_loop(alloc, total_len: np.ndarray, predicted: np.ndarray, concurrency: int,
                    on_event: Optional[Callable[[str, int, tuple], None]] = None,
                    on_epoch: Optional[Callable[[int, List[int], np.ndarray], None]] = None,
                    max_requests: Optional[int] = None) -> DriftResult:
    """Drive an allocator with a fixed-concurrency decode loop.

    `alloc` offers alloc(req, predicted) -> slab tuple (base, cap, pool, bucket)
    or None when memory is short, ensure(req, need) -> (slab tuple, migrated),
    or None when the Large Bucket cannot take the request (the request is then
    preempted: freed at its current length), commit(reqs, n_new) for a list of
    requests, free(req) and buckets() -> (tuple, epoch).  Request r is admitted with a prompt of
    max(1, total_len[r] // 4) tokens already in its slab, gains one token per
    step, and is freed when it reaches total_len[r]; the next request of the
    trace takes its place.  Steps in which nothing happens to the allocator are
    taken several at a time.  `on_event(kind, req, result)` sees every allocator
    answer; `on_epoch(epoch, live_reqs, live_lens)` is called whenever the
    boundary epoch changes.
    """
    n = int(total_len.shape[0]) if max_requests is None else min(int(total_len.shape[0]), max_requests)
    res = DriftResult()
    live: List[int] = []
    cur: List[int] = []
    cap: List[int] = []
    nxt = 0
    _, epoch = alloc.buckets()

    def admit():
        nonlocal nxt
        while nxt < n and len(live) < concurrency:
            r = nxt
            slab = alloc.alloc(r, int(predicted[r]))
            res.events += 1
            if on_event:
                on_event("alloc", r, slab)
            if slab is None:
                res.deferred += 1
                break
            prompt = max(1, int(total_len[r]) // 4)
            if prompt > slab[1]:
                ans = alloc.ensure(r, prompt)
                res.events += 1
                if on_event:
                    on_event("ensure", r, ans)
                if ans is None:
                    alloc.free(r)
                    res.events += 1
                    res.preempted += 1
                    nxt += 1
                    continue
                slab, mig = ans
                res.migrations += int(mig)
            alloc.commit([r], prompt)
            live.append(r)
            cur.append(prompt)
            cap.append(int(slab[1]))
            res.admitted += 1
            nxt += 1

    admit()
    while live:
        tot = total_len[np.asarray(live)]
        c = np.asarray(cur, dtype=np.int64)
        k_cap = np.asarray(cap, dtype=np.int64)
        to_finish = tot - c
        grow = k_cap < tot
        k = int(to_finish.min())
        if grow.any():
            k = min(k, int((k_cap - c)[grow].min()))
        if k <= 0:
            # some request stands at the end of its slab and still has tokens to produce
            dropped = []
            for j, r in enumerate(live):
                if cur[j] >= cap[j] and cur[j] < int(total_len[r]):
                    ans = alloc.ensure(r, cur[j] + 1)
                    res.events += 1
                    if on_event:
                        on_event("ensure", r, ans)
                    if ans is None:
                        alloc.free(r)
                        res.events += 1
                        res.preempted += 1
                        dropped.append(j)
                        continue
                    slab, mig = ans
                    res.migrations += int(mig)
                    cap[j] = int(slab[1])
            for j in reversed(dropped):
                del live[j], cur[j], cap[j]
            if dropped:
                admit()
            continue
        alloc.commit(list(live), k)
        for j in range(len(cur)):
            cur[j] += k
        res.steps += k
        done = [j for j, r in enumerate(live) if cur[j] >= int(total_len[r])]
        if done:
            for j in done:
                alloc.free(live[j])
                res.events += 1
                if on_event:
                    on_event("free", live[j], ())
            for j in reversed(done):
                del live[j], cur[j], cap[j]
            b, e = alloc.buckets()
            if e != epoch:
                epoch = e
                res.boundary_log.append((e, tuple(b)))
                if on_epoch:
                    on_epoch(e, list(live), np.asarray(cur, dtype=np.int64))
            admit()
    return res


# ---------------------------------------------------------------------------
# arrival trace for the admission simulator
# ---------------------------------------------------------------------------


def poisson_trace(seed: int, n: int, rate_per_s: float, law: str = "lognormal", noise_sigma: float = 0.3,
                  max_len: int = 16384, with_uncertainty: bool = False):
    """n requests arriving by a Poisson process of `rate_per_s`: rows of (arrival_ns, prompt,
    total, predicted, u_permille).  Totals follow the named length law (the stand-in for the
    request mix of the paper's evaluation, Section V), the prompt is a quarter of the total,
    the prediction is the total times a lognormal(0, noise_sigma) error.  With
    `with_uncertainty` the synthetic predictor also reports an uncertainty u in [0, 1] that
    grows with its (absolute, relative) error plus noise, so that a large u really does mark
    the requests whose prediction is poor; otherwise u = -1 (none)."""
    rng = _rng(seed)
    if law == "lognormal":
        total = lognormal_lengths(rng, n, 512, 0.8, 16, min(8192, max_len))
    elif law == "pareto":
        total = pareto_lengths(rng, n, 1.5, 32, max_len)
    else:
        raise ValueError(law)
    total = np.maximum(total, 2)
    prompt = np.clip(total // 4, 1, total - 1)
    predicted = np.minimum(noisy_prediction(rng, total, noise_sigma), max_len)
    arrival = np.cumsum(rng.exponential(1e9 / rate_per_s, size=n)).astype(np.int64)
    if with_uncertainty:
        rel = np.abs(predicted - total) / total
        u = np.clip(rel / (3 * noise_sigma) + rng.normal(0, 0.1, size=n), 0, 1)
        u_pm = np.rint(u * 1000).astype(np.int64)
    else:
        u_pm = np.full(n, -1, dtype=np.int64)
    return [(int(a), int(p), int(t), int(q), int(u)) for a, p, t, q, u in zip(arrival, prompt, total, predicted, u_pm)]
