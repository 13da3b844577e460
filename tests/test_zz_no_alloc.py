"""odma_decode_attention_static: decode attention for callers that cannot allocate GPU memory.

Some users of this library reach the attention call at a point where device allocation is
off the table: the serving process has handed the whole GPU to its own memory manager, or the
code runs as a plug-in of a framework that owns every allocation, or it sits on a path where
cudaMalloc's implicit device synchronisation is not acceptable.  For them the library offers
one entry point that keeps the partial results of split streams in a fixed array inside the
library image instead of scratch obtained from cudaMalloc, and that needs no device-backed
pool handle at all: a bookkeeping-only pool (created with no CUDA call) supplies the geometry,
odma_plan_host the plan, and the caller its own device copy of the plan.

The test drives exactly that flow and checks the result against the ordinary entry point
(odma_decode_attention) within the tolerances the other GPU tests use, on two calls in a row
(the second call finds the first call's partials still in the array).  It is collected last
so that a run that stops at the first failure has already run every other test, and it
depends on no state left by them.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from helpers import BF16_MAX_ABS, BF16_REL_L2, F32_MAX_ABS, Session, assert_close, host_pool, lib
from paper_2512_09427_b200 import workloads as wl

pytestmark = pytest.mark.gpu

LADDER = (16, 64, 256, 1024, 4096)


def _workload(lens, dtype, q_heads=28, kv_heads=4, head_dim=128):
    ctx = np.asarray(lens, dtype=np.int64)
    tokens = int(sum(min(b for b in LADDER if b >= L + 2) for L in lens) * 1.5) + 8192
    esz = 2 if dtype == torch.bfloat16 else 4
    return wl.Workload(name="noalloc", seed=4242, layers=2, q_heads=q_heads, kv_heads=kv_heads,
                       head_dim=head_dim, dtype=dtype, pool_bytes=tokens * 2 * 2 * kv_heads * head_dim * esz,
                       safety_pct=25, max_len=4096, context=ctx, predicted=ctx + 2, static_buckets=LADDER)


def _close(a, b, dtype):
    """The parity tests hold every entry point to max-abs 1e-2 / relative-L2 5e-3 (bf16) or
    1e-5 (fp32) of the fp64 checker.  Two results that each meet that bound can differ from
    one another by twice the max-abs bound (two bf16 roundings of values near 2 that fall on
    either side of a rounding boundary are one ulp = 2^-6 apart), so that is the elementwise
    bound between the two entry points; the relative-L2 bound is applied unchanged.  The
    static entry point is also checked against the checker itself at the plain tolerance."""
    x, y = a.double().cpu().numpy(), b.double().cpu().numpy()
    err = np.abs(x - y).max()
    rel = np.linalg.norm((x - y).ravel()) / max(np.linalg.norm(y.ravel()), 1e-300)
    if dtype == torch.bfloat16:
        assert err <= 2 * BF16_MAX_ABS and rel <= BF16_REL_L2, (err, rel)
    else:
        assert err <= 2 * F32_MAX_ABS, (err, rel)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_entry_point_matches_the_ordinary_one_twice_in_a_row(dtype):
    odma = lib()
    lens = [1, 63, 64, 200, 777, 2771]
    w = _workload(lens, dtype)
    # the ordinary path: a device pool, filled through the C ABI (the checker mirrors it)
    s = Session(w)
    assert s.pool.set_buckets(list(LADDER)) == s.ls.oracle.set_buckets(list(LADDER)) == 0
    reqs = list(range(w.batch))
    s.admit(reqs, w.predicted)
    s.append(reqs, [int(c) for c in w.context])
    s.decode_step(reqs, w.q_heads)                       # every request now holds context+1 tokens

    # the caller that cannot allocate: a bookkeeping-only pool replays the same reservations
    hp = host_pool(w, plan_ctas=37)
    assert hp.set_buckets(list(LADDER)) == 0
    for r in reqs:
        rc, slab = hp.alloc(r, int(w.predicted[r]))
        assert rc == odma.OK and slab[:2] == s.pool.get_slab(r)[1][:2]
        assert hp.commit_step([r], [s.lens[r]]) == 0
    rc, t, words = hp.plan_host(reqs, [0] * len(reqs))   # attend over what is there, append nothing
    assert rc == odma.OK and t.n_combine > 0             # some streams are split: the scratch array is used
    d_table = torch.tensor(words, dtype=torch.int32, device=s.dev)
    t.d_table = d_table.data_ptr()
    t_dev = s.tables(reqs, [0] * len(reqs))              # the ordinary path's own tables

    for call, layer in enumerate((0, 1)):
        q = s.queries(layer, reqs, w.q_heads, step=5 + call)
        want = torch.full_like(q, float("nan"))
        want_lse = torch.full((len(reqs), w.q_heads), float("nan"), dtype=torch.float32, device=s.dev)
        s.pool.decode_attention(layer, q.data_ptr(), w.q_heads, t_dev, want.data_ptr(), want_lse.data_ptr(), s.stream)
        got = torch.full_like(q, float("nan"))
        got_lse = torch.full_like(want_lse, float("nan"))
        rc = hp.decode_attention_static(s.mem.data_ptr(), layer, q.data_ptr(), w.q_heads, t, got.data_ptr(),
                                        got_lse.data_ptr(), s.stream)
        assert rc == odma.OK, odma.strerror(rc)
        torch.cuda.synchronize()
        assert s.pool.check_status(s.stream) == odma.OK
        assert torch.isfinite(got.float()).all() and torch.isfinite(got_lse).all()
        _close(got, want, dtype)
        assert (got_lse - want_lse).abs().max() <= (2e-2 if dtype == torch.bfloat16 else 1e-5)
        ref, _, _ = s.oracle_out(layer, reqs, q, w.q_heads)      # and against the fp64 checker
        assert_close(got, ref, dtype, f"static call {call}")


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    odma = lib()
    w = _workload([100, 200], torch.bfloat16, q_heads=32, kv_heads=2)       # 16 query heads per KV head
    hp = host_pool(w, max_group=16)
    assert hp.set_buckets(list(LADDER)) == 0
    for r in range(2):
        assert hp.alloc(r, int(w.predicted[r]))[0] == odma.OK
        assert hp.commit_step([r], [int(w.context[r])]) == 0
    rc, t, words = hp.plan_host([0, 1], [0, 0])
    assert rc == odma.OK
    dev = torch.device("cuda:0")
    mem = torch.zeros(w.pool_bytes, dtype=torch.uint8, device=dev)
    d_table = torch.tensor(words, dtype=torch.int32, device=dev)
    t.d_table = d_table.data_ptr()
    q = torch.zeros(2, 32, 128, dtype=torch.bfloat16, device=dev)
    out = torch.zeros_like(q)
    rc = hp.decode_attention_static(mem.data_ptr(), 0, q.data_ptr(), 32, t, out.data_ptr())
    assert rc == odma.ERR_TOO_LARGE and "scratch" in odma.strerror(rc)
    # a misaligned pool base is an argument error, not a fault
    assert hp.decode_attention_static(mem.data_ptr() + 16, 0, q.data_ptr(), 32, t, out.data_ptr()) == odma.ERR_INVALID
