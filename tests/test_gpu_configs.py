"""GPU parity on the full-size evaluation workloads (configs 3, 4 and 5).

The pools are too large to mirror in the CPU checker's own store, so the checker's inputs are
regenerated on the CPU from the seeded counter-based generator (every K/V element is a pure
function of (seed, layer, request, kind, index)) for the sampled requests, and the allocator
is compared in lock step at every call as everywhere else.
"""
import numpy as np
import pytest
import torch

from helpers import Session, assert_close, lib, warm_up
from oracle import oracle as ora
from paper_2512_09427_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[1, 2], ids=["tcgen05", "mma_sync"])
def decode_kernel(request):
    """Every test of this module runs once on each bf16 tensor-core decode kernel."""
    import helpers
    helpers.CFG_DEFAULTS["decode_kernel"] = request.param
    yield request.param
    helpers.CFG_DEFAULTS.clear()


def checker_out(w, layer, reqs, lens, q):
    """fp64 attention of `reqs` (KV lengths `lens`) on `layer` from regenerated inputs."""
    Ks = [wl.kv_rows(w.seed, layer, r, wl.KIND_K, 0, L, w.kv_heads, w.head_dim, w.dtype) for r, L in zip(reqs, lens)]
    Vs = [wl.kv_rows(w.seed, layer, r, wl.KIND_V, 0, L, w.kv_heads, w.head_dim, w.dtype) for r, L in zip(reqs, lens)]
    out, lse, _ = ora.decode_attention(q.cpu(), Ks, Vs, w.q_heads, w.kv_heads, w.head_dim, ora.dtype_code(w.dtype),
                                       want_lse=True)
    return out, lse


def check_sample(s, w, res, reqs, sample, what):
    pos = {r: i for i, r in enumerate(reqs)}
    idx = torch.tensor([pos[r] for r in sample], device=s.dev)
    for layer, (out, lse, q) in res.items():
        assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all(), what
        ref, ref_lse = checker_out(w, layer, sample, [s.lens[r] for r in sample], q[idx])
        err = assert_close(out[idx], ref, w.dtype, f"{what} layer {layer}")
        assert np.abs(lse[idx].double().cpu().numpy() - ref_lse).max() <= 2e-2
        print(what, "layer", layer, "max_abs %.2e rel_l2 %.2e" % err)


def test_config3_full_pool_noisy_predictions_and_migrations():
    """40 GB, 28-layer pool; 256 Pareto-length requests admitted with noisy predictions, so
    some start in the Large Bucket and some migrate; one decode step with append; every
    request checked on three of the layers."""
    w = wl.config3()
    s = Session(w, mirror_kv=False)
    warm_up(s.ls, w.warmup_lengths)
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    layers = [0, 13, 27]
    s.append(reqs, [int(c) for c in w.context], layers=layers)
    res = s.decode_step(reqs, w.q_heads, layers=layers)
    st = s.ls.check_stats()
    assert st["migrations"] > 0 and st["used_live"] == int(w.context.sum()) + w.batch
    large = [r for r in reqs if s.pool.get_slab(r)[1][2] == 1]
    assert large, "some requests must sit in the Large Bucket"
    check_sample(s, w, res, reqs, reqs, "config3")
    print("config3: migrations", st["migrations"], "in the Large Bucket", len(large),
          "utilisation %.3f" % (st["used_live"] / st["reserved_live"]))


def test_config5_long_contexts_split_streams_and_paged_ablation():
    """Batch 32, contexts U[16384, 32768] (two of the 28 layers, the full per-layer size of
    1.6 GB): every stream is split over several CTAs.  All 32 requests against the checker on
    both layers; the page-16 copy (pages shuffled) must give the same bits as the slab layout."""
    odma = lib()
    base = wl.config5()
    w = wl.scaled(base, layers=2, pool_bytes=base.pool_bytes // 14)
    s = Session(w, mirror_kv=False)
    warm_up(s.ls, w.warmup_lengths)
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    res = s.decode_step(reqs, w.q_heads)
    t = s.last_tables
    assert t.n_combine >= w.batch * w.kv_heads // 2           # long streams: most are split
    check_sample(s, w, res, reqs, reqs, "config5")
    # page-16 ablation on identical inputs
    host_len = [s.lens[r] for r in reqs]
    max_pages = max(-(-L // 16) for L in host_len)
    n_pages = sum(-(-L // 16) for L in host_len) + 11
    page_bytes = w.layers * 2 * w.kv_heads * 16 * w.head_dim * 2
    pages = torch.empty(n_pages * page_bytes, dtype=torch.uint8, device=s.dev)
    pages.view(torch.int16).fill_(0x7FC0)
    ptab = torch.zeros(len(reqs) * max_pages, dtype=torch.int32, device=s.dev)
    paged = odma.Paged(s.pool, pages.data_ptr(), pages.numel())
    t0 = s.tables(reqs, [0] * len(reqs))
    paged.build(t0, host_len, 950905, ptab.data_ptr(), max_pages, s.stream)
    for layer, (out, lse, q) in res.items():
        out_p = torch.full_like(out, float("nan"))
        lse_p = torch.full_like(lse, float("nan"))
        paged.decode_attention(layer, q.data_ptr(), w.q_heads, t0, ptab.data_ptr(), max_pages, out_p.data_ptr(),
                               lse_p.data_ptr(), s.stream)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == 0
        assert torch.equal(out_p, out) and torch.equal(lse_p, lse)


class DeviceLoop:
    """Allocator face for workloads.run_closed_loop that also writes every committed token's
    K/V rows into the device pool (layer 0), so the pool holds real caches when a boundary
    epoch arrives."""

    def __init__(self, s):
        self.s, self.len = s, {}

    def alloc(self, req, predicted):
        slab = self.s.ls.alloc(req, predicted)
        if slab is not None:
            self.len[req] = 0
        return slab

    def ensure(self, req, need):
        return self.s.ls.ensure(req, need)

    def commit(self, reqs, n_new):
        s, w = self.s, self.s.w
        reqs = [int(r) for r in reqs]
        t = s.tables(reqs, [n_new] * len(reqs))
        a = [self.len[r] for r in reqs]
        b = [x + n_new for x in a]
        k = wl.kv_rows_batch(w.seed, 0, reqs, wl.KIND_K, a, b, w.kv_heads, w.head_dim, w.dtype, s.dev)
        v = wl.kv_rows_batch(w.seed, 0, reqs, wl.KIND_V, a, b, w.kv_heads, w.head_dim, w.dtype, s.dev)
        s.pool.append_kv(0, t, k.data_ptr(), v.data_ptr(), s.stream)
        s.ls.commit(reqs, n_new)
        for r in reqs:
            self.len[r] += n_new

    def free(self, req):
        self.s.ls.free(req)
        del self.len[req]

    def buckets(self):
        return self.s.ls.buckets()


def test_config4_drift_stream_attention_at_boundary_epochs():
    """The drifting request stream through a device pool, allocator in lock step with the
    checker at every event; at each boundary recalibration the live batch (128 requests at
    whatever lengths and wherever their slabs ended up, migrated ones included) is attended
    and a sample of it compared with the checker."""
    w = wl.config4(noisy=True)
    s = Session(w, mirror_kv=False)
    assert s.pool.set_buckets(list(w.static_buckets)) == s.ls.oracle.set_buckets(list(w.static_buckets)) == 0
    loop = DeviceLoop(s)
    seen = []

    def on_epoch(epoch, live, lens):
        reqs = [int(r) for r in live]
        assert [loop.len[r] for r in reqs] == [int(x) for x in lens]
        t = s.tables(reqs, [0] * len(reqs))
        q = s.queries(0, reqs, w.q_heads, step=epoch)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev)
        s.pool.decode_attention(0, q.data_ptr(), w.q_heads, t, out.data_ptr(), lse.data_ptr(), s.stream)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == 0
        assert torch.isfinite(out.float()).all()
        order = np.argsort(lens)
        pick = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), 0, len(reqs) - 1})
        migrated = [i for i, r in enumerate(reqs) if s.pool.get_slab(r)[1][2] == 1][:2]
        pick = sorted(set(pick + migrated))
        idx = torch.tensor(pick, device=s.dev)
        sample = [reqs[i] for i in pick]
        ref, ref_lse = checker_out(w, 0, sample, [loop.len[r] for r in sample], q[idx])
        err = assert_close(out[idx], ref, w.dtype, f"config4 epoch {epoch}")
        assert np.abs(lse[idx].double().cpu().numpy() - ref_lse).max() <= 2e-2
        seen.append((epoch, len(reqs), int(lens.sum()), len(migrated), err))

    res = wl.run_closed_loop(loop, w.context, w.predicted, w.extra["concurrency"], on_epoch=on_epoch,
                             max_requests=1600)
    assert res.admitted == 1600 and len(seen) == 1600 // w.refresh
    st = s.ls.check_stats()
    assert st["completed"] == 1600 and st["migrations"] > 0
    print("config4:", seen, "migrations", st["migrations"],
          "utilisation %.3f" % (st["sum_len_completed"] / st["sum_cap_completed"]))


def test_config2_in_the_benchmarks_own_launch_configuration(decode_kernel):
    """bench.py's set-up and step for config 2 (rotating KV copies, odma_decode_step with the
    append and the merge inside the decode kernel, plan reused from step to step): outputs of
    sampled requests on two of the copies against the checker, and the appended rows in place."""
    import bench
    odma = lib()
    w, step_layers, copies = bench.pick_workload("config2")
    sd = bench.SlabDecode(w, step_layers, torch.device("cuda:0"), decode_kernel=decode_kernel)
    bounds, epoch = sd.learn_boundaries()
    assert len(bounds) == 4 and epoch == 10
    sd.admit_and_fill()
    q, kn, vn, out = sd.make_inputs()
    t = odma.Tables()
    for i in range(2 * copies):                    # every copy twice: the second pass reuses the plan
        sd.step(i, q, kn, vn, out, t)
    torch.cuda.synchronize()
    assert sd.pool.check_status(sd.stream) == odma.OK
    assert t.n_ctas == 148 and t.kv_tokens == int((w.context + 1).sum())
    order = np.argsort(w.context)
    sample = sorted({int(order[0]), int(order[len(order) // 2]), int(order[-1]), 0, w.batch - 1})
    idx = torch.tensor(sample, device=sd.dev)
    for layer in (0, copies - 1):
        ref, _ = checker_out(w, layer, sample, [int(w.context[r]) + 1 for r in sample], q[layer][idx])
        err = assert_close(out[layer][idx], ref, w.dtype, f"bench configuration, copy {layer}")
        print("config2 as benchmarked, copy", layer, "max_abs %.2e rel_l2 %.2e" % err)
        # the step's token sits behind each sampled request's context in the slab
        T = sd.pool.get_stats()["total_tokens"]
        arr = sd.mem.view(w.dtype)[: w.layers * 2 * T * w.kv_heads * w.head_dim].view(w.layers * 2, T * w.kv_heads, w.head_dim)
        for r in sample:
            rc, slab, ln = sd.pool.get_slab(r)
            base, cap = slab[0], slab[1]
            for kv, new in ((0, kn), (1, vn)):
                for h in range(w.kv_heads):
                    row = base * w.kv_heads + h * cap + int(w.context[r])
                    assert torch.equal(arr[layer * 2 + kv][row], new[layer][r, h])


def test_config2_benchmark_pattern_300_overlapping_steps_bit_identical():
    """What bench.py times: the config-2 step repeated on three rotating KV copies (layers of one
    pool) with no synchronisation, so that consecutive launches overlap.  The step on a copy is
    the same computation every pass (the same token re-appended at the same position), so the
    results of passes 1 to 99 must be equal bit for bit; passes 0 and 1 are checked against the
    checker."""
    odma = lib()
    w = wl.config2(layers=3)
    s = Session(w, mirror_kv=False, decode_kernel=0)
    warm_up(s.ls, w.warmup_lengths)
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    for r in reqs:
        s.ls.ensure(r, s.lens[r] + 1)
    L = w.layers
    q = torch.stack([s.queries(l, reqs, w.q_heads, 0) for l in range(L)]).contiguous()
    kn = torch.stack([torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]) for l in range(L)]).contiguous()
    vn = torch.stack([torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]) for l in range(L)]).contiguous()
    passes = 100
    outs = torch.full((passes, L) + tuple(q.shape[1:]), float("nan"), dtype=q.dtype, device=s.dev)
    lses = torch.full((passes, L, len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev)
    torch.cuda.synchronize()
    for k in range(passes):                      # no synchronisation inside this loop
        for l in range(L):
            s.pool.decode_step(l, 1, w.q_heads, reqs, q[l].data_ptr(), kn[l].data_ptr(), vn[l].data_ptr(),
                               outs[k, l].data_ptr(), lses[k, l].data_ptr(), s.stream)
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == odma.OK
    for r in reqs:
        s.lens[r] += 1
    sample = reqs[::7]
    pos = torch.tensor(sample, device=s.dev)
    # The run's very first launch has nothing to chain to and may be served by the other kernel, so
    # pass 0 is checked on its own and pass 1 is the one the rest must equal.
    for l in range(L):
        ref, ref_lse = checker_out(w, l, sample, [s.lens[r] for r in sample], q[l][pos])
        for k in (0, 1):
            assert_close(outs[k, l][pos], ref, w.dtype, f"config2 copy {l} pass {k}")
            assert np.abs(lses[k, l][pos].double().cpu().numpy() - ref_lse).max() <= 2e-2
    differ = (outs[1:].view(torch.int16) != outs[1].view(torch.int16)).flatten(1).any(dim=1)
    assert not bool(differ.any()), ("passes that differ from pass 1", differ.nonzero().flatten().tolist()[:10])
    assert bool((lses[1:] == lses[1]).all())
