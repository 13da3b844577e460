"""GPU parity of the 8-bit (E4M3) slab variant: stored codes bit for bit, attention over them
against the fp64 checker, through the C ABI."""
import numpy as np
import pytest
import torch

from helpers import BF16_MAX_ABS, BF16_REL_L2, Session, attention_errors, lib
from paper_2512_09427_b200 import workloads as wl

pytestmark = pytest.mark.gpu

RAGGED = [1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 95, 96, 97, 127, 128, 129, 500, 1000, 2771]


def small(lens, layers=1, q_heads=28, kv_heads=4, seed=91):
    ladder = (16, 64, 256, 1024, 4096)
    ctx = np.asarray(lens, dtype=np.int64)
    tokens = int(sum(min(b for b in ladder if b >= L + 1) for L in lens) * 1.5) + 8192
    w = wl.Workload(name="small", seed=seed, layers=layers, q_heads=q_heads, kv_heads=kv_heads, head_dim=128,
                    dtype=torch.bfloat16, pool_bytes=tokens * layers * 2 * kv_heads * 128 * 2, safety_pct=25,
                    max_len=4096, context=ctx, predicted=ctx + 8, static_buckets=ladder)
    return wl.with_e4m3(w)


def start(w, fill=0x7F7F, **cfg):
    """Session with the contexts appended (through odma_append_kv, which quantises)."""
    s = Session(w, fill=fill, **cfg)          # 0x7F7F: every untouched byte is the NaN code
    if w.static_buckets:
        assert s.pool.set_buckets(list(w.static_buckets)) == s.ls.oracle.set_buckets(list(w.static_buckets)) == 0
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    pre = [r for r in reqs if w.context[r] > 0]
    if pre:
        s.append(pre, [int(w.context[r]) for r in pre])
    return s, reqs


def check(s, layer, reqs, q, out, lse, what):
    """The stated tolerance: the bf16 bounds, the absolute one following the size of the values."""
    ref, ref_lse, _ = s.oracle_out(layer, reqs, q, s.w.q_heads)
    assert torch.isfinite(out.float()).all(), what
    err, rel = attention_errors(out, ref)
    vmax = 448.0 * s.v_scale[layer]
    assert err <= BF16_MAX_ABS * max(1.0, vmax / 4.0) and rel <= BF16_REL_L2, (what, err, rel)
    if lse is not None:
        l = lse.double().cpu().numpy()
        assert np.isfinite(l).all() and np.abs(l - ref_lse).max() <= 2e-2, what
    return err, rel


def check_codes(s, reqs, layers):
    for r in reqs:
        for l in layers:
            k_ref, v_ref = s.kv.gathered(r, l)
            assert np.array_equal(s.pool_rows(l, 0, r).cpu().numpy(), k_ref), ("K codes", r, l)
            assert np.array_equal(s.pool_rows(l, 1, r).cpu().numpy(), v_ref), ("V codes", r, l)


def test_append_stores_the_checkers_codes_and_nothing_else():
    w = small([L - 1 for L in RAGGED], layers=2)
    s, reqs = start(w)
    pre = [r for r in reqs if w.context[r] > 0]
    check_codes(s, pre, range(w.layers))
    # several tokens at once behind existing ones, and values beyond the format's range (saturation)
    s.append(pre[:5], [3, 1, 7, 2, 16], scale=200.0)
    check_codes(s, pre[:5], range(w.layers))
    touched = torch.zeros(s.T * w.kv_heads, dtype=torch.bool, device=s.dev)
    for r in pre:
        rc, slab, ln = s.pool.get_slab(r)
        for h in range(w.kv_heads):
            b = slab[0] * w.kv_heads + h * slab[1]
            touched[b: b + ln] = True
    arr = s.mem[: w.layers * 2 * s.T * w.kv_heads * 128].view(w.layers * 2, s.T * w.kv_heads, 128)
    assert (arr[:, ~touched] == 0x7F).all()


@pytest.mark.parametrize("fused", [1, 0])
@pytest.mark.parametrize("ctas", [0, 1, 23])
def test_ragged_lengths_span_tiles_key_groups_and_splits(ctas, fused):
    w = small([L - 1 for L in RAGGED])
    s, reqs = start(w, plan_ctas=ctas, fused_combine=fused)
    for step in range(2):
        res = s.decode_step(reqs, w.q_heads, step=step)
        t = s.last_tables
        if ctas == 23:
            assert t.n_combine > 0
        out, lse, q = res[0]
        e = check(s, 0, reqs, q, out, lse, f"ragged ctas={ctas} fused={fused} step={step}")
    check_codes(s, reqs, [0])
    print("e4m3 ragged", ctas, fused, e)


@pytest.mark.parametrize("span", [1, 0], ids=["one_launch", "launch_per_layer"])
@pytest.mark.parametrize("ctas", [0, 5])
def test_fused_steps_over_chained_layers(ctas, span):
    """odma_decode_step: the new token is quantised by the decode kernel, used as its code's value
    and written into the slab; layers chain.  Three steps back to back without a host sync."""
    odma = lib()
    lens = [0, 1, 31, 32, 63, 64, 129, 700, 1500, 2771]
    w = small(lens, layers=4)
    s, reqs = start(w, plan_ctas=ctas, span_layers=span)
    steps, NL = 3, w.layers
    qs = [torch.stack([s.queries(l, reqs, w.q_heads, k) for l in range(NL)]).contiguous() for k in range(steps)]
    kns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_K, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs])
                        for l in range(NL)]).contiguous() for k in range(steps)]
    vns = [torch.stack([torch.cat([s.rows(l, r, wl.KIND_V, s.lens[r] + k, s.lens[r] + k + 1) for r in reqs])
                        for l in range(NL)]).contiguous() for k in range(steps)]
    outs = [torch.full_like(qs[0], float("nan")) for _ in range(steps)]
    lses = [torch.full((NL, len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev) for _ in range(steps)]
    for r in reqs:
        s.ls.ensure(r, s.lens[r] + steps)
    torch.cuda.synchronize()
    t = odma.Tables()
    for k in range(steps):
        s.pool.decode_step(0, NL, w.q_heads, reqs, qs[k].data_ptr(), kns[k].data_ptr(), vns[k].data_ptr(),
                           outs[k].data_ptr(), lses[k].data_ptr(), s.stream, t)
        s.ls.commit(reqs, 1)
    torch.cuda.synchronize()
    assert s.pool.check_status(s.stream) == odma.OK
    for k in range(steps):
        for l in range(NL):
            for i, r in enumerate(reqs):
                s.kv.append(r, l, kns[k][l, i:i + 1], vns[k][l, i:i + 1])
            check(s, l, reqs, qs[k][l], outs[k][l], lses[k][l], f"step {k} layer {l}")
    for r in reqs:
        s.lens[r] += steps
    check_codes(s, reqs, range(NL))


def test_scores_scaled_by_eight_and_tiny_queries():
    """Peaked softmax (the reference maximum is raised and the accumulator rescaled in tensor
    memory) and queries 2^-20 of the usual size (the per-row power of two of the split)."""
    w = small([200, 1000, 2771, 64])
    s, reqs = start(w, plan_ctas=7)
    res = s.decode_step(reqs, w.q_heads, scale=8.0)
    out, lse, q = res[0]
    check(s, 0, reqs, q, out, lse, "x8")
    res = s.decode_step(reqs, w.q_heads, step=1, scale=2.0 ** -20)
    out, lse, q = res[0]
    check(s, 0, reqs, q, out, lse, "tiny q")


def test_other_group_sizes():
    for q_heads, kv_heads in [(8, 8), (16, 2), (4, 4), (14, 2)]:
        w = small([5, 100, 640, 1500], q_heads=q_heads, kv_heads=kv_heads)
        s, reqs = start(w)
        res = s.decode_step(reqs, w.q_heads)
        out, lse, q = res[0]
        check(s, 0, reqs, q, out, lse, f"group {q_heads}/{kv_heads}")


def test_migration_moves_codes():
    w = small([10, 60, 700])
    s, reqs = start(w)                               # slabs of 64, 256 and 1024 tokens
    before = s.pool.get_stats()["migrations"]
    s.append(reqs, [60, 200, 5])                     # 70 > 64 and 260 > 256: two migrate
    assert s.pool.get_stats()["migrations"] == before + 2
    check_codes(s, reqs, [0])
    res = s.decode_step(reqs, w.q_heads)
    out, lse, q = res[0]
    check(s, 0, reqs, q, out, lse, "after migration")


def test_unsupported_shapes_and_calls_are_refused():
    odma = lib()
    mem = torch.zeros(1 << 24, dtype=torch.uint8, device="cuda:0")
    for head_dim in (64, 96):
        with pytest.raises(odma.OdmaError):
            odma.Pool(mem.data_ptr(), mem.numel(), 1, 2, head_dim, odma.DTYPE_FP8_E4M3)
    cfg = odma.config_default()
    cfg.decode_kernel = odma.DECODE_MMA_SYNC
    with pytest.raises(odma.OdmaError):
        odma.Pool(mem.data_ptr(), mem.numel(), 1, 2, 128, odma.DTYPE_FP8_E4M3, cfg)
    pool = odma.Pool(mem.data_ptr(), mem.numel(), 1, 2, 128, odma.DTYPE_FP8_E4M3)
    with pytest.raises(odma.OdmaError):
        pool.set_kv_scales([0.0], [1.0])
    with pytest.raises(odma.OdmaError):
        pool.set_kv_scales([1.0], [float("inf")])
    with pytest.raises(odma.OdmaError):
        odma.Paged(pool, mem.data_ptr(), 1 << 20)
    bf = odma.Pool(mem.data_ptr(), mem.numel(), 1, 2, 128, odma.DTYPE_BF16)
    with pytest.raises(odma.OdmaError):
        bf.set_kv_scales([1.0], [1.0])


def test_config2_shape_parity_and_config5_shape_sampled():
    """The evaluation shapes on 8-bit slabs: config 2 whole (one layer), and the first eight
    requests of config 5 (16-32 k tokens each: streams cut into pieces that are merged)."""
    from helpers import warm_up
    c5 = wl.config5()
    c5 = wl.scaled(c5, layers=1, pool_bytes=c5.pool_bytes // 28 // 3, context=c5.context[:8], predicted=c5.predicted[:8])
    for w in (wl.with_e4m3(wl.config2()), wl.with_e4m3(c5)):
        s = Session(w)
        if w.static_buckets:
            s.pool.set_buckets(list(w.static_buckets)); s.ls.oracle.set_buckets(list(w.static_buckets))
        if w.warmup_lengths is not None:
            warm_up(s.ls, w.warmup_lengths)
        reqs = list(range(w.batch))
        s.admit(reqs, w.predicted)
        s.append(reqs, [int(x) for x in w.context], layers=[0])
        res = s.decode_step(reqs, w.q_heads, layers=[0])
        out, lse, q = res[0]
        e = check(s, 0, reqs, q, out, lse, w.name)
        print(w.name, e, "split streams:", s.last_tables.n_combine)
