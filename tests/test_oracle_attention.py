"""Pins for the CPU checker's attention (oracle/odma_oracle.c, part 1).

None of these retype the checker's formula: they compare it with a library
routine (torch fp64 scaled_dot_product_attention), with closed forms, with
invariants of softmax attention, and with a 50-digit evaluation on tiny inputs.
Each is chosen so that a plausible slip (wrong scale, wrong KV-head mapping,
transposed operand, dropped max-subtraction, bf16 widened wrongly) fails.
"""
import math

import mpmath
import numpy as np
import pytest
import torch

from oracle import oracle as ora


def _rand(shape, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(dtype)


def _sdpa_fp64(q, k, v):
    """q [Hq,D], k/v [L,Hkv,D] -> library attention in fp64 with KV heads repeated per group."""
    hq, hkv = q.shape[0], k.shape[1]
    g = hq // hkv
    qd = q.double().unsqueeze(1)                                   # [Hq,1,D]
    kd = k.double().permute(1, 0, 2).repeat_interleave(g, dim=0)   # [Hq,L,D]
    vd = v.double().permute(1, 0, 2).repeat_interleave(g, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(qd, kd, vd)
    s = (qd @ kd.transpose(1, 2)).squeeze(1) / math.sqrt(q.shape[1])
    return o.squeeze(1).numpy(), torch.logsumexp(s, dim=-1).numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("hq,hkv,d", [(28, 4, 128), (2, 1, 64), (8, 8, 32), (6, 2, 16)])
def test_matches_library_sdpa_fp64(dtype, hq, hkv, d):
    code = ora.dtype_code(dtype)
    lens = [1, 7, 64, 65, 333]
    q = _rand((len(lens), hq, d), dtype, 1)
    K = [_rand((L, hkv, d), dtype, 10 + i) for i, L in enumerate(lens)]
    V = [_rand((L, hkv, d), dtype, 20 + i) for i, L in enumerate(lens)]
    out, lse, _ = ora.decode_attention(q, K, V, hq, hkv, d, code, want_lse=True)
    for i in range(len(lens)):
        ref, ref_lse = _sdpa_fp64(q[i], K[i], V[i])
        np.testing.assert_allclose(out[i], ref, rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[i], ref_lse, rtol=0, atol=1e-12)


def test_large_scores_are_stable():
    # scores around +-400: a missing max-subtraction overflows exp()
    hq, hkv, d, L = 4, 2, 64, 50
    q = _rand((1, hq, d), torch.float32, 3) * 20
    K = [_rand((L, hkv, d), torch.float32, 4) * 20]
    V = [_rand((L, hkv, d), torch.float32, 5)]
    out, lse, _ = ora.decode_attention(q, K, V, hq, hkv, d, ora.F32, want_lse=True)
    ref, ref_lse = _sdpa_fp64(q[0], K[0], V[0])
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    np.testing.assert_allclose(out[0], ref, atol=1e-11)
    np.testing.assert_allclose(lse[0], ref_lse, atol=1e-9)


def test_single_key_returns_its_value_exactly():
    hq, hkv, d = 6, 3, 32
    for dtype in (torch.float32, torch.bfloat16):
        q = _rand((1, hq, d), dtype, 6)
        k = _rand((1, hkv, d), dtype, 7)
        v = _rand((1, hkv, d), dtype, 8)
        out, _, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.dtype_code(dtype))
        for h in range(hq):
            assert np.array_equal(out[0, h], v[0, h // 2].double().numpy())


def test_zero_query_gives_mean_of_values():
    hq, hkv, d, L = 4, 2, 16, 37
    q = torch.zeros(1, hq, d)
    k = _rand((L, hkv, d), torch.float32, 9)
    v = _rand((L, hkv, d), torch.float32, 10)
    out, lse, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32, want_lse=True)
    for h in range(hq):
        np.testing.assert_allclose(out[0, h], v[:, h // 2].double().mean(0).numpy(), atol=1e-14)
        assert abs(lse[0, h] - math.log(L)) < 1e-14


def test_equal_keys_give_mean_and_constant_values_pass_through():
    hq, hkv, d, L = 4, 1, 16, 11
    q = _rand((1, hq, d), torch.float32, 11)
    k = _rand((1, hkv, d), torch.float32, 12).expand(L, hkv, d).contiguous()
    v = _rand((L, hkv, d), torch.float32, 13)
    out, _, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32)
    for h in range(hq):
        np.testing.assert_allclose(out[0, h], v[:, 0].double().mean(0).numpy(), atol=1e-14)
    k2 = _rand((L, hkv, d), torch.float32, 14)
    vconst = _rand((1, hkv, d), torch.float32, 15).expand(L, hkv, d).contiguous()
    out2, _, _ = ora.decode_attention(q, [k2], [vconst], hq, hkv, d, ora.F32)
    for h in range(hq):
        np.testing.assert_allclose(out2[0, h], vconst[0, 0].double().numpy(), atol=1e-14)


def test_two_keys_closed_form_pins_scale_and_sign():
    # q = (a,0,..), k0 = (c,0,..), k1 = 0: weights are sigmoid(+-a*c/sqrt(D)).
    d = 64
    a, c = 3.0, 2.0
    q = torch.zeros(1, 1, d)
    q[0, 0, 0] = a
    k = torch.zeros(2, 1, d)
    k[0, 0, 0] = c
    v = torch.zeros(2, 1, d)
    v[0, 0, 0] = 1.0
    v[1, 0, 1] = 1.0
    out, w, lse = ora.attention_weights(q[0], k, v, 0, 1, 1, d, ora.F32)
    z = a * c / math.sqrt(d)
    w0 = 1.0 / (1.0 + math.exp(-z))
    assert abs(w[0] - w0) < 1e-15 and abs(w[1] - (1 - w0)) < 1e-15
    assert abs(out[0] - w0) < 1e-15 and abs(out[1] - (1 - w0)) < 1e-15
    assert abs(lse - math.log(math.exp(z) + 1.0)) < 1e-14


def test_dominant_key_selects_its_value():
    hq, hkv, d, L = 2, 1, 64, 40
    q = torch.zeros(1, hq, d)
    q[0, :, 0] = 8.0
    k = torch.zeros(L, hkv, d)
    k[17, 0, 0] = 60.0     # score 8*60/8 = 60 above all others (0)
    v = _rand((L, hkv, d), torch.float32, 16)
    out, _, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32)
    np.testing.assert_allclose(out[0, 0], v[17, 0].double().numpy(), atol=1e-20 + 40 * math.exp(-60) * 5)


def test_kv_head_mapping_is_h_div_group():
    # Every KV head kappa has its own dominant key at position kappa; query head h must
    # return V[h div g] at that position.  A wrong mapping (h mod Hkv, transposed) fails.
    hq, hkv, d, L = 12, 4, 32, 9
    g = hq // hkv
    q = torch.zeros(1, hq, d)
    q[0, :, 0] = 10.0
    k = torch.zeros(L, hkv, d)
    for kap in range(hkv):
        k[kap, kap, 0] = 100.0
    v = _rand((L, hkv, d), torch.float32, 17)
    out, _, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32)
    for h in range(hq):
        np.testing.assert_allclose(out[0, h], v[h // g, h // g].double().numpy(), atol=1e-12)


def test_weights_sum_to_one_and_are_positive():
    hq, hkv, d, L = 7, 1, 128, 500
    q = _rand((hq, d), torch.bfloat16, 18)
    k = _rand((L, hkv, d), torch.bfloat16, 19)
    v = _rand((L, hkv, d), torch.bfloat16, 20)
    for h in range(hq):
        _, w, _ = ora.attention_weights(q, k, v, h, hq, hkv, d, ora.BF16)
        assert (w > 0).all()
        assert abs(w.sum() - 1.0) < 1e-13


def test_permuting_keys_with_their_values_changes_nothing():
    hq, hkv, d, L = 4, 2, 64, 97
    q = _rand((1, hq, d), torch.float32, 21)
    k = _rand((L, hkv, d), torch.float32, 22)
    v = _rand((L, hkv, d), torch.float32, 23)
    perm = torch.randperm(L, generator=torch.Generator().manual_seed(5))
    a, _, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32)
    b, _, _ = ora.decode_attention(q, [k[perm].contiguous()], [v[perm].contiguous()], hq, hkv, d, ora.F32)
    np.testing.assert_allclose(a, b, atol=1e-14)
    # permuting keys WITHOUT their values must change the result (a K/V mix-up is visible)
    c, _, _ = ora.decode_attention(q, [k[perm].contiguous()], [v], hq, hkv, d, ora.F32)
    assert np.abs(a - c).max() > 1e-3


def test_tiny_inputs_against_50_digit_arithmetic():
    mpmath.mp.dps = 50
    hq, hkv, d, L = 2, 1, 4, 5
    q = _rand((1, hq, d), torch.float32, 24)
    k = _rand((L, hkv, d), torch.float32, 25)
    v = _rand((L, hkv, d), torch.float32, 26)
    out, lse, _ = ora.decode_attention(q, [k], [v], hq, hkv, d, ora.F32, want_lse=True)
    for h in range(hq):
        qq = mpmath.matrix([mpmath.mpf(float(x)) for x in q[0, h]])
        kk = mpmath.matrix([[mpmath.mpf(float(x)) for x in k[j, 0]] for j in range(L)])
        vv = mpmath.matrix([[mpmath.mpf(float(x)) for x in v[j, 0]] for j in range(L)])
        scores = (kk * qq) / mpmath.sqrt(d)
        z = mpmath.fsum(mpmath.e ** s for s in scores)
        o = vv.T * mpmath.matrix([mpmath.e ** s / z for s in scores])
        for j in range(d):
            assert abs(mpmath.mpf(out[0, h, j]) - o[j]) < mpmath.mpf("1e-15")
        assert abs(mpmath.mpf(lse[0, h]) - mpmath.log(z)) < mpmath.mpf("1e-14")


def test_bf16_is_widened_exactly():
    # bf16 patterns 0x3F80 = 1.0, 0xC000 = -2.0, 0x3DCD ~ 0.10009765625
    bits = np.array([0x3F80, 0xC000, 0x3DCD, 0x0000], dtype=np.uint16)
    v = bits.reshape(1, 1, 4)
    q = np.zeros((1, 1, 4), dtype=np.uint16)
    out, _, _ = ora.decode_attention(q, [v.copy()], [v], 1, 1, 4, ora.BF16)
    assert out[0, 0].tolist() == [1.0, -2.0, 0.10009765625, 0.0]


@pytest.mark.parametrize("chunk", [1, 16, 64, 100])
def test_split_and_merge_equals_dense(chunk):
    # the log-sum-exp merge of independent pieces is exact (up to fp64 rounding)
    hq, hkv, d, L = 4, 2, 32, 203
    q = _rand((hq, d), torch.float32, 27) * 3
    k = _rand((L, hkv, d), torch.float32, 28) * 3
    v = _rand((L, hkv, d), torch.float32, 29)
    for h in range(hq):
        dense, _, _ = ora.attention_weights(q, k, v, h, hq, hkv, d, ora.F32)
        merged = ora.attention_chunked(q, k, v, h, hq, hkv, d, ora.F32, chunk)
        np.testing.assert_allclose(merged, dense, atol=1e-12)


def test_kv_store_keeps_append_order():
    st = ora.KVStore(1, 2, 8, ora.F32)
    a = _rand((3, 2, 8), torch.float32, 30)
    b = _rand((1, 2, 8), torch.float32, 31)
    st.append(5, 0, a, a * 2)
    st.append(5, 0, b, b * 2)
    k, v = st.gathered(5, 0)
    assert st.length(5) == 4
    assert np.array_equal(k, torch.cat([a, b]).numpy()) and np.array_equal(v, 2 * torch.cat([a, b]).numpy())


def test_prefill_chunk_is_causal_attention():
    """The chunk form against an independent library's masked attention in fp64: token j of the
    chunk sees the context and the chunk's tokens up to itself."""
    rng = np.random.default_rng(21)
    Hq, Hkv, D, ctx, chunk = 4, 2, 16, 11, 7
    K = rng.standard_normal((ctx + chunk, Hkv, D)).astype(np.float32)
    V = rng.standard_normal((ctx + chunk, Hkv, D)).astype(np.float32)
    q = rng.standard_normal((chunk, Hq, D)).astype(np.float32)
    st = ora.KVStore(1, Hkv, D, ora.F32)
    st.append(5, 0, K[:ctx], V[:ctx])
    st.append(5, 0, K[ctx:], V[ctx:])
    out, lse = ora.prefill_attention(st, 0, [5], [chunk], q, Hq)
    qt = torch.from_numpy(q).double().permute(1, 0, 2)                        # [Hq, chunk, D]
    kt = torch.from_numpy(K).double().permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)
    vt = torch.from_numpy(V).double().permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)
    mask = torch.arange(ctx + chunk)[None, :] <= (ctx + torch.arange(chunk))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask).permute(1, 0, 2).numpy()
    assert np.max(np.abs(out - ref)) < 1e-12
    # a fresh prompt's first token attends itself alone
    st2 = ora.KVStore(1, Hkv, D, ora.F32)
    st2.append(1, 0, K[:3], V[:3])
    o2, l2 = ora.prefill_attention(st2, 0, [1], [3], q[:3], Hq)
    for h in range(Hq):
        assert np.allclose(o2[0, h], V[0, h // (Hq // Hkv)], rtol=0, atol=1e-15)
