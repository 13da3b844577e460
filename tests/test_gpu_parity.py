"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU checker."""
import numpy as np
import pytest
import torch

from conftest import read_golden
from helpers import (BF16_MAX_ABS, BF16_REL_L2, Session, assert_close, attention_errors, lib)
from paper_2512_09427_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[(1, 2), (1, 1), (2, 0)], ids=["tcgen05", "tcgen05_late_readout", "mma_sync"])
def decode_kernel(request):
    """Every test of this module runs once on each bf16 tensor-core decode kernel, on the tcgen05
    kernel with both orders of reading an item's result out."""
    import helpers
    helpers.CFG_DEFAULTS["decode_kernel"], helpers.CFG_DEFAULTS["readout"] = request.param
    yield request.param[0]
    helpers.CFG_DEFAULTS.clear()

RAGGED = [1, 15, 16, 17, 63, 64, 65, 127, 128, 129, 500, 1000, 2771]


def qwen_small(lens, layers=1, q_heads=28, kv_heads=4, head_dim=128, dtype=torch.bfloat16, seed=77):
    """A Qwen-shaped workload over explicit context lengths with one static bucket ladder."""
    ladder = (16, 64, 256, 1024, 4096)
    ctx = np.asarray(lens, dtype=np.int64)
    tokens = int(sum(min(b for b in ladder if b >= L + 1) for L in lens) * 1.5) + 8192
    esz = 2 if dtype == torch.bfloat16 else 4
    return wl.Workload(name="small", seed=seed, layers=layers, q_heads=q_heads, kv_heads=kv_heads,
                       head_dim=head_dim, dtype=dtype, pool_bytes=tokens * layers * 2 * kv_heads * head_dim * esz,
                       safety_pct=25, max_len=4096, context=ctx, predicted=ctx + 1, static_buckets=ladder)


def run_decode(w, cfg_over=None, fill=None, scale=1.0, layers=None):
    s = Session(w, fill=fill, **(cfg_over or {}))
    if w.static_buckets:
        assert s.pool.set_buckets(list(w.static_buckets)) == s.ls.oracle.set_buckets(list(w.static_buckets)) == 0
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    if pre:
        s.append(pre, [int(w.context[r]) for r in pre], scale=scale)
    res = s.decode_step(reqs, w.q_heads, layers=layers, scale=scale)
    return s, reqs, res


def check_all(s, reqs, res, what=""):
    worst = (0.0, 0.0)
    for layer, (out, lse, q) in res.items():
        ref, ref_lse, _ = s.oracle_out(layer, reqs, q, s.w.q_heads)
        assert torch.isfinite(out.float()).all(), what
        e = assert_close(out, ref, s.w.dtype, f"{what} layer {layer}")
        worst = max(worst, e)
        l = lse.double().cpu().numpy()
        assert np.isfinite(l).all()
        assert np.abs(l - ref_lse).max() <= (2e-2 if s.w.dtype == torch.bfloat16 else 1e-5), what
    return worst


# ---------------------------------------------------------------------------------------------


@pytest.mark.parametrize("variant", ["a", "b"])
def test_config1_allocation_append_and_attention(variant):
    w = wl.config1(variant)
    s, reqs, res = run_decode(w, fill=0x7B7B)       # sentinel-filled pool: canary for stray writes
    # slab tables equal the hand-computed ones
    rows = [r for r in read_golden("config1_alloc.txt") if r[0] == "1" + variant and r[1] == "ensure"]
    for _, _, req, _, base, cap, pl, bucket, _ in rows:
        rc, slab, ln = s.pool.get_slab(int(req))
        assert slab[:4] == (int(base), int(cap), int(pl), int(bucket))
        assert ln == int(w.context[int(req)]) + 1
    if variant == "b":
        assert s.pool.get_stats()["migrations"] == 1
    check_all(s, reqs, res, "config1" + variant)
    # the pool, read back through the documented layout, holds exactly the appended rows ...
    touched = torch.zeros(s.T * w.kv_heads, dtype=torch.bool, device=s.dev)
    for r in reqs:
        k_ref, v_ref = s.kv.gathered(r, 0)
        assert np.array_equal(s.pool_rows(0, 0, r).cpu().numpy(), k_ref)
        assert np.array_equal(s.pool_rows(0, 1, r).cpu().numpy(), v_ref)
        rc, slab, ln = s.pool.get_slab(r)
        touched[slab[0] * w.kv_heads: slab[0] * w.kv_heads + ln] = True
    # ... and nothing else was written (the migrated request's old slab [64,128) still holds its copy)
    arr = s.mem.view(torch.int16)[: 2 * s.T * w.kv_heads * w.head_dim * 2].view(2, s.T * w.kv_heads, -1)
    if variant == "b":
        touched[64:128] = True
    assert (arr[:, ~touched] == 0x7B7B).all()


@pytest.mark.parametrize("fused", [1, 0])
@pytest.mark.parametrize("ctas", [0, 1, 23])
def test_bf16_ragged_lengths_span_tiles_and_splits(ctas, fused):
    w = qwen_small([L - 1 for L in RAGGED])
    s, reqs, res = run_decode(w, cfg_over={"plan_ctas": ctas, "fused_combine": fused})
    t = s.last_tables
    if ctas == 23:
        assert t.n_combine > 0                      # some streams were split and merged
    if ctas == 1:
        assert t.n_combine == 0
    err = check_all(s, reqs, res, f"ragged ctas={ctas} fused={fused}")
    # a second step on the same pool: the split-stream counters were left at zero
    res2 = s.decode_step(reqs, w.q_heads, step=1)
    check_all(s, reqs, res2, f"ragged second step ctas={ctas} fused={fused}")
    print("bf16 ragged", ctas, fused, err)


@pytest.mark.parametrize("ctas", [1, 3])
def test_repeated_launches_with_many_items_per_cta_are_bit_identical(ctas):
    """52 items on one CTA (or three): the query ring wraps six times and its slots are refilled
    the moment they are released, merge buffers and stages are reused back to back.  The kernel
    is deterministic, so every repeat of the launch must give the bits of the first one (which is
    checked against the checker); a slot refilled while a consumer still reads it shows up here
    as a few rows that differ in some repeats."""
    w = qwen_small([L - 1 for L in RAGGED])
    s, reqs, res = run_decode(w, cfg_over={"plan_ctas": ctas})
    check_all(s, reqs, res, f"many items per CTA, ctas={ctas}")
    out0, lse0, q = res[0]
    t = s.last_tables
    assert t.n_items >= 52 and t.n_ctas == ctas
    for rep in range(24):
        out = torch.full_like(out0, float("nan"))
        lse = torch.full_like(lse0, float("nan"))
        s.pool.decode_attention(0, q.data_ptr(), w.q_heads, t, out.data_ptr(), lse.data_ptr(), s.stream)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == 0
        assert torch.equal(out, out0) and torch.equal(lse, lse0), f"repeat {rep} differs"


@pytest.mark.parametrize("ctas", [1, 3])
def test_repeated_fused_steps_with_many_items_per_cta_are_bit_identical(ctas):
    """The same stress through odma_decode_step with the append fused in: the query slots then
    also carry each stream's new K/V rows.  The step is repeated without committing lengths, so
    every repeat appends the same rows at the same place and must give the same bits."""
    odma = lib()
    w = qwen_small([L - 1 for L in RAGGED])
    w = wl.scaled(w, predicted=w.context + 8)
    s = Session(w, plan_ctas=ctas)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    s.append(pre, [int(w.context[r]) for r in pre])
    for r in reqs:
        s.ls.ensure(r, s.lens[r] + 1)
    q = s.queries(0, reqs, w.q_heads, 0).contiguous()
    kn = torch.cat([s.rows(0, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
    vn = torch.cat([s.rows(0, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
    out0 = None
    for rep in range(25):
        out = torch.full_like(q, float("nan"))
        s.pool.decode_step(0, 1, w.q_heads, reqs, q.data_ptr(), kn.data_ptr(), vn.data_ptr(), out.data_ptr(), 0, s.stream)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == odma.OK
        if out0 is None:
            out0 = out
            for i, r in enumerate(reqs):
                s.kv.append(r, 0, kn[i:i + 1], vn[i:i + 1])
            ref, _, _ = s.oracle_out(0, reqs, q, w.q_heads)
            assert_close(out0, ref, w.dtype, f"fused step, many items per CTA, ctas={ctas}")
        else:
            assert torch.equal(out, out0), f"repeat {rep} differs"
    s.ls.commit(reqs, 1)
    for r in reqs:
        s.lens[r] += 1
        k_ref, v_ref = s.kv.gathered(r, 0)
        assert np.array_equal(s.pool_rows(0, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
        assert np.array_equal(s.pool_rows(0, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


def test_migration_copy_then_fused_step_without_a_host_sync():
    """A request outgrows its slab: the migration copy and the decode step that reads the
    copied rows are enqueued back to back.  The decode kernel must not read slab rows before the
    copy kernel ahead of it has completed (it may only do so behind another decode kernel)."""
    odma = lib()
    lens = [63, 64, 200, 1024]
    w = qwen_small(lens)
    w = wl.scaled(w, predicted=w.context)            # slabs exactly full: 64 and 1024 overflow on the next token
    s = Session(w, plan_ctas=4)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    q = s.queries(0, reqs, w.q_heads, 0).contiguous()
    kn = torch.cat([s.rows(0, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
    vn = torch.cat([s.rows(0, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
    out = torch.full_like(q, float("nan"))
    torch.cuda.synchronize()
    migrated = sum(s.ls.ensure(r, s.lens[r] + 1)[1] for r in reqs)     # launches the copies, no sync
    s.pool.decode_step(0, 1, w.q_heads, reqs, q.data_ptr(), kn.data_ptr(), vn.data_ptr(), out.data_ptr(), 0, s.stream)
    torch.cuda.synchronize()
    assert migrated == 2 and s.pool.check_status(s.stream) == odma.OK
    s.ls.commit(reqs, 1)
    for i, r in enumerate(reqs):
        s.kv.append(r, 0, kn[i:i + 1], vn[i:i + 1])
        s.lens[r] += 1
    ref, _, _ = s.oracle_out(0, reqs, q, w.q_heads)
    assert_close(out, ref, w.dtype, "migration then fused step")
    for r in reqs:
        k_ref, v_ref = s.kv.gathered(r, 0)
        assert np.array_equal(s.pool_rows(0, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)


def test_fused_and_separate_combine_agree_bit_for_bit():
    w = qwen_small([L - 1 for L in RAGGED] + [4000])
    outs = []
    for fused in (1, 0):
        s, reqs, res = run_decode(w, cfg_over={"plan_ctas": 23, "fused_combine": fused})
        assert s.last_tables.n_combine > 0
        outs.append(res[0])
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("span", [1, 0], ids=["one_launch", "launch_per_layer"])
@pytest.mark.parametrize("ctas", [1, 3, 0])
def test_late_and_immediate_readout_agree_bit_for_bit(ctas, span, decode_kernel):
    """The tcgen05 kernel reads an item's result out at once or under the next item of the same half
    of the CTA: the same arithmetic in another order of hand-overs, so every output bit, every
    log-sum-exp and every appended row agree.  Many short items per CTA (up to 60 per half and
    layer), items of no tile at all, split streams, three layers, two steps without a host sync."""
    if decode_kernel != 1:
        pytest.skip("tcgen05 kernel only")
    odma = lib()
    lens = [0, 1, 2, 15, 16, 17, 40, 63, 64, 65, 100, 127, 128, 129, 130, 200, 31, 33, 5, 7, 9, 11, 300, 2771, 70, 90, 3, 0, 64, 128]
    w = qwen_small(lens, layers=3)
    w = wl.scaled(w, predicted=w.context + 8)
    got = []
    for readout in (odma.READOUT_LATE, odma.READOUT_AT_ONCE):
        s = Session(w, plan_ctas=ctas, span_layers=span, readout=readout)
        s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
        reqs = list(range(w.batch))
        s.admit(reqs, w.predicted)
        pre = [r for r in reqs if w.context[r] > 0]
        s.append(pre, [int(w.context[r]) for r in pre])
        steps, NL = 2, w.layers
        qs = [torch.stack([s.queries(l, reqs, w.q_heads, k) for l in range(NL)]).contiguous() for k in range(steps)]
        kns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs])
                            for l in range(NL)]).contiguous() for k in range(steps)]
        vns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs])
                            for l in range(NL)]).contiguous() for k in range(steps)]
        outs = [torch.full_like(qs[0], float("nan")) for _ in range(steps)]
        lses = [torch.full((NL, len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev) for _ in range(steps)]
        torch.cuda.synchronize()
        t = odma.Tables()
        for k in range(steps):
            s.pool.decode_step(0, NL, w.q_heads, reqs, qs[k].data_ptr(), kns[k].data_ptr(), vns[k].data_ptr(),
                               outs[k].data_ptr(), lses[k].data_ptr(), s.stream, t)
            s.ls.commit(reqs, 1)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == odma.OK
        if ctas == 0:
            assert t.n_combine > 0
        if readout == odma.READOUT_LATE:                    # and the late order against the checker
            for k in range(steps):
                for l in range(NL):
                    for i, r in enumerate(reqs):
                        s.kv.append(r, l, kns[k][l, i:i + 1], vns[k][l, i:i + 1])
                    ref, ref_lse, _ = s.oracle_out(l, reqs, qs[k][l], w.q_heads)
                    assert_close(outs[k][l], ref, w.dtype, f"late step {k} layer {l}")
                    assert np.abs(lses[k][l].double().cpu().numpy() - ref_lse).max() <= 2e-2
        for r in reqs:
            s.lens[r] += steps
        rows = [s.pool_rows(l, kind, r).clone() for l in range(NL) for kind in (0, 1) for r in reqs]
        got.append((outs, lses, rows))
    (o1, l1, r1), (o2, l2, r2) = got
    for a, b in zip(o1 + l1 + r1, o2 + l2 + r2):
        assert torch.equal(a, b)


def test_bf16_multi_layer_and_second_step():
    w = qwen_small([40, 300, 64, 1, 130], layers=3)
    s, reqs, res = run_decode(w)
    check_all(s, reqs, res, "3 layers")
    res2 = s.decode_step(reqs, w.q_heads, step=1)
    check_all(s, reqs, res2, "second step")
    for layer in range(3):
        for r in reqs:
            k_ref, v_ref = s.kv.gathered(r, layer)
            assert np.array_equal(s.pool_rows(layer, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
            assert np.array_equal(s.pool_rows(layer, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


@pytest.mark.parametrize("q_heads,kv_heads,head_dim", [(24, 2, 128), (24, 2, 64), (8, 8, 64), (14, 2, 128), (4, 4, 128)])
def test_bf16_other_group_sizes_and_head_dims(q_heads, kv_heads, head_dim):
    w = qwen_small([5, 63, 64, 200, 777], q_heads=q_heads, kv_heads=kv_heads, head_dim=head_dim)
    s, reqs, res = run_decode(w, cfg_over={"max_group": 16, "plan_ctas": 5})
    check_all(s, reqs, res, f"{q_heads}/{kv_heads}/{head_dim}")


@pytest.mark.parametrize("dtype,q_heads,kv_heads,head_dim", [
    (torch.float32, 28, 4, 128), (torch.float32, 2, 1, 64), (torch.float32, 6, 2, 32),
    (torch.bfloat16, 40, 2, 128), (torch.bfloat16, 6, 2, 32)])
def test_generic_path_fp32_and_wide_groups(dtype, q_heads, kv_heads, head_dim):
    w = qwen_small([0, 31, 32, 100, 257, 900], q_heads=q_heads, kv_heads=kv_heads, head_dim=head_dim, dtype=dtype)
    s, reqs, res = run_decode(w, cfg_over={"max_group": 32, "plan_ctas": 6})
    check_all(s, reqs, res, f"generic {dtype} {q_heads}/{kv_heads}/{head_dim}")


def test_nan_poisoned_pool_changes_nothing():
    lens = [L - 1 for L in RAGGED]
    w = qwen_small(lens)
    s0, reqs, res0 = run_decode(w)
    s1, _, res1 = run_decode(w, fill=0x7FC0)        # every untouched bf16 is a NaN
    for layer in res0:
        assert torch.isfinite(res1[layer][0].float()).all()
        assert torch.equal(res0[layer][0], res1[layer][0])
        assert torch.equal(res0[layer][1], res1[layer][1])


def test_scores_scaled_by_eight_stay_stable():
    w = qwen_small([100, 1000, 64])
    s, reqs, res = run_decode(w, scale=8.0 ** 0.5)       # q and k both scaled: scores x 8
    for layer, (out, lse, q) in res.items():
        ref, ref_lse, _ = s.oracle_out(layer, reqs, q, w.q_heads)
        assert torch.isfinite(out.float()).all()
        err, rel = attention_errors(out, ref)
        # softmax is nearly one-hot here: bf16 rounding of P matters less, of the output more
        assert err <= 2e-2 and rel <= 1e-2, (err, rel)


def test_migration_keeps_the_cache_and_attention_right():
    # slabs exactly full before the step: every request migrates to the Large Bucket
    w = qwen_small([16, 64, 256], layers=2)
    w = wl.scaled(w, predicted=w.context.copy())
    s, reqs, res = run_decode(w)
    assert s.pool.get_stats()["migrations"] == 3
    for r in reqs:
        assert s.pool.get_slab(r)[1][2] == 1
    check_all(s, reqs, res, "migrated")


def test_paged_copy_gives_the_same_attention():
    odma = lib()
    lens = [L - 1 for L in RAGGED]
    w = qwen_small(lens, layers=2)
    s, reqs, res = run_decode(w, cfg_over={"plan_ctas": 9})
    t = s.last_tables
    host_len = [s.lens[r] for r in reqs]
    max_pages = max(-(-L // 16) for L in host_len)
    n_pages = sum(-(-L // 16) for L in host_len) + 37
    page_bytes = w.layers * 2 * w.kv_heads * 16 * w.head_dim * 2
    pages = torch.zeros(n_pages * page_bytes, dtype=torch.uint8, device=s.dev)
    ptab = torch.zeros(len(reqs) * max_pages, dtype=torch.int32, device=s.dev)
    paged = odma.Paged(s.pool, pages.data_ptr(), pages.numel())
    for seed in (0, 12345):
        pages.view(torch.int16).fill_(0x7FC0)
        paged.build(t, host_len, seed, ptab.data_ptr(), max_pages, s.stream)
        ids = ptab.view(len(reqs), max_pages).cpu().numpy()
        used = np.concatenate([ids[i, : -(-L // 16)] for i, L in enumerate(host_len)])
        assert len(set(used.tolist())) == len(used) and used.max() < n_pages
        if seed == 0:
            assert used.tolist() == list(range(len(used)))
        else:
            assert used.tolist() != sorted(used.tolist())
        for layer, (out, lse, q) in res.items():
            out_p = torch.full_like(out, float("nan"))
            lse_p = torch.full_like(lse, float("nan"))
            paged.decode_attention(layer, q.data_ptr(), w.q_heads, t, ptab.data_ptr(), max_pages,
                                   out_p.data_ptr(), lse_p.data_ptr(), s.stream)
            torch.cuda.synchronize()
            assert s.pool.check_status(s.stream) == 0
            assert torch.equal(out_p, out) and torch.equal(lse_p, lse)     # same arithmetic, other layout


def test_read_probe_and_bounded_wait_selftest():
    odma = lib()
    w = qwen_small([100, 1000, 64])
    s, reqs, res = run_decode(w)
    s.pool.read_probe(0, w.q_heads, s.last_tables, s.stream)
    assert s.pool.check_status(s.stream) == odma.OK
    # a wait that nothing will ever satisfy gives up and reports, and the context lives on
    assert s.pool.selftest_timeout(20, s.stream) == odma.OK
    assert s.pool.check_status(s.stream) == odma.ERR_TIMEOUT
    assert s.pool.check_status(s.stream) == odma.OK
    res2 = s.decode_step(reqs, w.q_heads, step=1)
    check_all(s, reqs, res2, "after the timeout self-test")


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_from_host_buffers_matches_the_device_path(pinned):
    """Page-locked buffers are read and written in place by the kernel (no copy); pageable ones
    are staged through device scratch.  Same result either way, and the new rows are in the slab."""
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    w = qwen_small([10, 200, 64, 999])
    s = Session(w)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    for r in reqs:
        s.ls.ensure(r, s.lens[r] + 1)
    q = pin(s.queries(0, reqs, w.q_heads).cpu())
    k_new = pin(torch.cat([s.rows(0, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]).cpu())
    v_new = pin(torch.cat([s.rows(0, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]).cpu())
    out = pin(torch.full_like(q, float("nan")))
    assert q.is_pinned() == pinned and out.is_pinned() == pinned
    s.pool.decode_step_host(0, w.q_heads, reqs, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                            out.data_ptr(), s.stream)
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == 0
    for i, r in enumerate(reqs):
        s.kv.append(r, 0, k_new[i:i + 1], v_new[i:i + 1])
    ref, _, _ = s.oracle_out(0, reqs, q, w.q_heads)
    assert_close(out, ref, w.dtype, "host step")
    s.ls.commit(reqs, 1)                              # pool_rows reads up to the committed length
    for i, r in enumerate(reqs):                      # the step's rows sit behind each context
        assert torch.equal(s.pool_rows(0, 0, r)[-1].cpu(), k_new[i]) and torch.equal(s.pool_rows(0, 1, r)[-1].cpu(), v_new[i])


@pytest.mark.parametrize("fused_append", [1, 0])
def test_decode_step_with_the_append_inside_the_decode_kernel(fused_append, decode_kernel):
    """odma_decode_step: the new token is taken from k_new / v_new by the decode kernel itself
    (never read from the slab) and written into the slab for later steps.  Lengths chosen so
    that some streams consist of the new token alone, some end a tile exactly, some are split."""
    odma = lib()
    lens = [0, 1, 63, 64, 127, 128, 500, 2771]
    w = qwen_small(lens, layers=2)
    s = Session(w, fill=0x7FC0, plan_ctas=19, fused_append=fused_append)     # untouched rows are NaN
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    s.append(pre, [int(w.context[r]) for r in pre])
    for step in range(2):
        for r in reqs:
            s.ls.ensure(r, s.lens[r] + 1)
        q = torch.stack([s.queries(l, reqs, w.q_heads, step) for l in range(w.layers)]).contiguous()
        kn = torch.stack([torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]) for l in range(w.layers)]).contiguous()
        vn = torch.stack([torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]) for l in range(w.layers)]).contiguous()
        out = torch.full_like(q, float("nan"))
        lse = torch.full((w.layers, len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev)
        t = odma.Tables()
        s.pool.profile_enable(True)
        s.pool.decode_step(0, w.layers, w.q_heads, reqs, q.data_ptr(), kn.data_ptr(), vn.data_ptr(), out.data_ptr(),
                           lse.data_ptr(), s.stream, t)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == odma.OK
        assert s.pool.profile_read(odma.K_APPEND)[1] == (0 if fused_append else w.layers)
        # with the append fused in, both layers of the step are one launch of the tcgen05 kernel
        assert s.pool.profile_read(odma.K_DECODE)[1] == (1 if fused_append and decode_kernel == 1 else w.layers)
        s.pool.profile_enable(False)
        assert t.n_combine > 0
        s.ls.commit(reqs, 1)
        for l in range(w.layers):
            for i, r in enumerate(reqs):
                s.kv.append(r, l, kn[l, i:i + 1], vn[l, i:i + 1])
        for r in reqs:
            s.lens[r] += 1
        for l in range(w.layers):
            ref, ref_lse, _ = s.oracle_out(l, reqs, q[l], w.q_heads)
            assert torch.isfinite(out[l].float()).all() and torch.isfinite(lse[l]).all()
            assert_close(out[l], ref, w.dtype, f"fused step {step} layer {l}")
            assert np.abs(lse[l].double().cpu().numpy() - ref_lse).max() <= 2e-2
            for r in reqs:                      # the slab now holds the new rows, bit for bit
                k_ref, v_ref = s.kv.gathered(r, l)
                assert np.array_equal(s.pool_rows(l, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
                assert np.array_equal(s.pool_rows(l, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


def test_many_fused_steps_reuse_the_plan_and_then_replan():
    """36 consecutive decode steps of one batch through odma_decode_step: the plan of step 0
    serves until the batch has grown by 32 tokens per request (lengths ride in the kernel
    arguments, streams cross tile boundaries on the way), then a fresh plan is made."""
    odma = lib()
    lens = [30, 62, 63, 100, 127, 500, 1000]
    w = qwen_small(lens)
    w = wl.scaled(w, predicted=w.context + 64)
    s = Session(w, plan_ctas=11)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    t = odma.Tables()
    plans = []
    for step in range(36):
        q = s.queries(0, reqs, w.q_heads, step).contiguous()
        kn = torch.cat([s.rows(0, r, wl.KIND_K, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
        vn = torch.cat([s.rows(0, r, wl.KIND_V, s.lens[r], s.lens[r] + 1) for r in reqs]).contiguous()
        out = torch.full_like(q, float("nan"))
        s.pool.decode_step(0, 1, w.q_heads, reqs, q.data_ptr(), kn.data_ptr(), vn.data_ptr(), out.data_ptr(), 0,
                           s.stream, t)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == odma.OK
        plans.append((t.n_items, t.kv_tokens))
        s.ls.commit(reqs, 1)
        for i, r in enumerate(reqs):
            s.kv.append(r, 0, kn[i:i + 1], vn[i:i + 1])
            s.lens[r] += 1
        if step in (0, 1, 17, 31, 32, 33, 35):
            ref, _, _ = s.oracle_out(0, reqs, q, w.q_heads)
            assert_close(out, ref, w.dtype, f"step {step}")
    assert [kv for _, kv in plans] == [sum(lens) + w.batch * (k + 1) for k in range(36)]
    for r in reqs:                                  # every appended row reached the slab
        k_ref, v_ref = s.kv.gathered(r, 0)
        assert np.array_equal(s.pool_rows(0, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
        assert np.array_equal(s.pool_rows(0, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


def test_back_to_back_steps_on_one_layer_without_host_syncs():
    """Steps enqueued back to back on the same layer: each kernel starts (and requests its first
    tiles) while its predecessor, which is still appending a row to every stream, drains.  All
    outputs and every appended row must come out as if the steps had run one at a time."""
    odma = lib()
    lens = [70, 129, 200, 640, 1500, 3000]
    w = qwen_small(lens)
    w = wl.scaled(w, predicted=w.context + 48)
    s = Session(w, plan_ctas=13)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    steps = 24
    qs = [s.queries(0, reqs, w.q_heads, k).contiguous() for k in range(steps)]
    kns = [torch.cat([s.rows(0, r, wl.KIND_K, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]).contiguous() for k in range(steps)]
    vns = [torch.cat([s.rows(0, r, wl.KIND_V, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]).contiguous() for k in range(steps)]
    outs = [torch.full_like(qs[0], float("nan")) for _ in range(steps)]
    torch.cuda.synchronize()
    for k in range(steps):                       # no synchronisation inside this loop
        s.pool.decode_step(0, 1, w.q_heads, reqs, qs[k].data_ptr(), kns[k].data_ptr(), vns[k].data_ptr(),
                           outs[k].data_ptr(), 0, s.stream)
        s.ls.commit(reqs, 1)
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == odma.OK
    for k in range(steps):
        for i, r in enumerate(reqs):
            s.kv.append(r, 0, kns[k][i:i + 1], vns[k][i:i + 1])
        ref, _, _ = s.oracle_out(0, reqs, qs[k], w.q_heads)
        assert_close(outs[k], ref, w.dtype, f"step {k}")
    for r in reqs:
        s.lens[r] += steps
        k_ref, v_ref = s.kv.gathered(r, 0)
        assert np.array_equal(s.pool_rows(0, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
        assert np.array_equal(s.pool_rows(0, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


@pytest.mark.parametrize("span", [1, 0], ids=["one_launch", "launch_per_layer"])
@pytest.mark.parametrize("ctas", [0, 5])
def test_layers_of_one_step_run_chained_without_host_syncs(ctas, span):
    """odma_decode_step over six layers, three steps enqueued back to back: the kernel of layer
    l > 0 does not wait for the kernel of layer l - 1 (other K/V arrays, other outputs, the other
    scratch set), so kernels of neighbouring layers run side by side.  Every layer of every
    step against the checker, and every appended row in place."""
    odma = lib()
    lens = [0, 40, 64, 129, 700, 1500, 2771]
    w = qwen_small(lens, layers=6)
    w = wl.scaled(w, predicted=w.context + 8)
    s = Session(w, plan_ctas=ctas, span_layers=span)      # all six layers in one launch, or a chained launch each
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    s.append(pre, [int(w.context[r]) for r in pre])
    steps, NL = 3, w.layers
    qs = [torch.stack([s.queries(l, reqs, w.q_heads, k) for l in range(NL)]).contiguous() for k in range(steps)]
    kns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]) for l in range(NL)]).contiguous()
           for k in range(steps)]
    vns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]) for l in range(NL)]).contiguous()
           for k in range(steps)]
    outs = [torch.full_like(qs[0], float("nan")) for _ in range(steps)]
    lses = [torch.full((NL, len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev) for _ in range(steps)]
    torch.cuda.synchronize()
    t = odma.Tables()
    for k in range(steps):                       # no synchronisation inside this loop
        s.pool.decode_step(0, NL, w.q_heads, reqs, qs[k].data_ptr(), kns[k].data_ptr(), vns[k].data_ptr(),
                           outs[k].data_ptr(), lses[k].data_ptr(), s.stream, t)
        s.ls.commit(reqs, 1)
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == odma.OK
    if ctas == 0:
        assert t.n_combine > 0
    for k in range(steps):
        for l in range(NL):
            for i, r in enumerate(reqs):
                s.kv.append(r, l, kns[k][l, i:i + 1], vns[k][l, i:i + 1])
            ref, ref_lse, _ = s.oracle_out(l, reqs, qs[k][l], w.q_heads)
            assert torch.isfinite(outs[k][l].float()).all()
            assert_close(outs[k][l], ref, w.dtype, f"step {k} layer {l}")
            assert np.abs(lses[k][l].double().cpu().numpy() - ref_lse).max() <= 2e-2
    for r in reqs:
        s.lens[r] += steps
        for l in range(NL):
            k_ref, v_ref = s.kv.gathered(r, l)
            assert np.array_equal(s.pool_rows(l, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
            assert np.array_equal(s.pool_rows(l, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)


@pytest.mark.parametrize("fused", [1, 0])
def test_profile_counts_launches(fused):
    odma = lib()
    w = qwen_small([100, 1000, 64])
    s, reqs, _ = run_decode(w, cfg_over={"plan_ctas": 16, "fused_combine": fused})
    s.pool.profile_enable(True)
    s.decode_step(reqs, w.q_heads, step=1)
    ms, n = s.pool.profile_read(odma.K_DECODE)
    assert n == 1 and ms > 0
    assert s.pool.profile_read(odma.K_APPEND)[1] == 1
    assert s.last_tables.n_combine > 0
    assert s.pool.profile_read(odma.K_COMBINE)[1] == (0 if fused else 1)     # fused: merged in the decode kernel
    s.pool.profile_enable(False)


def test_config2_full_size_parity():
    """The benchmark workload itself: 64 requests, log-normal contexts, learned quartile buckets."""
    from helpers import warm_up
    w = wl.config2()
    s = Session(w)
    warm_up(s.ls, w.warmup_lengths)
    bounds, epoch = s.ls.buckets()
    assert epoch == 10 and len(bounds) == 4
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    res = s.decode_step(reqs, w.q_heads)
    err = check_all(s, reqs, res, "config2")
    st = s.ls.check_stats()
    print("config2 parity", err, "buckets", bounds, "reserved", st["reserved_live"], "used", st["used_live"])


@pytest.mark.parametrize("kernel", [0, 1], ids=["auto", "tcgen05"])
def test_consecutive_steps_on_different_layers_overlap_and_stay_right(kernel):
    """Single-layer odma_decode_step calls issued back to back on changing layers (the pattern of
    a multi-layer model, and of the benchmark's rotating KV copies): each runs without waiting
    for the one before; where a round ends on the layer the next round starts with, that launch
    must wait.  Twelve calls without a host synchronisation, every one against the checker, every
    appended row in place."""
    odma = lib()
    lens = [0, 40, 64, 129, 700, 1500, 2771]
    w = qwen_small(lens, layers=4)
    w = wl.scaled(w, predicted=w.context + 8)
    s = Session(w, plan_ctas=11, decode_kernel=kernel)
    s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    s.append(pre, [int(w.context[r]) for r in pre])
    rounds = [[0, 1, 2, 3], [3, 0, 2, 1], [1, 3, 0, 2]]             # token k goes to every layer in round k
    calls = []
    for k, order in enumerate(rounds):
        for l in order:
            q = s.queries(l, reqs, w.q_heads, 10 + k)
            kn = torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]).contiguous()
            vn = torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs]).contiguous()
            out = torch.full_like(q, float("nan"))
            lse = torch.full((len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev)
            calls.append((k, l, q, kn, vn, out, lse))
    for r in reqs:
        s.ls.ensure(r, s.lens[r] + len(rounds))
    torch.cuda.synchronize()
    for i, (k, l, q, kn, vn, out, lse) in enumerate(calls):        # no synchronisation inside this loop
        s.pool.decode_step(l, 1, w.q_heads, reqs, q.data_ptr(), kn.data_ptr(), vn.data_ptr(), out.data_ptr(),
                           lse.data_ptr(), s.stream)
        if i % 4 == 3:
            s.ls.commit(reqs, 1)                                    # the round's token, host bookkeeping only
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == odma.OK
    for (k, l, q, kn, vn, out, lse) in calls:
        for i, r in enumerate(reqs):
            s.kv.append(r, l, kn[i:i + 1], vn[i:i + 1])
        ref, ref_lse, _ = s.oracle_out(l, reqs, q, w.q_heads)
        assert torch.isfinite(out.float()).all()
        assert_close(out, ref, w.dtype, f"round {k} layer {l}")
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() <= 2e-2
    for r in reqs:
        s.lens[r] += len(rounds)
        for l in range(w.layers):
            k_ref, v_ref = s.kv.gathered(r, l)
            assert np.array_equal(s.pool_rows(l, 0, r).view(torch.int16).cpu().numpy().view(np.uint16), k_ref)
            assert np.array_equal(s.pool_rows(l, 1, r).view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
