"""Pins of the checker's E4M3 arithmetic (oracle/odma_oracle.c): the format's published special
values, torch's float8_e4m3fn as an independent implementation of widening and of
round-to-nearest-even, and closed forms of attention over a quantised store."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "e4m3_format.txt")


def _rows():
    vals, rounds = [], []
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        if line[0] == "r":
            rounds.append((float(line[1]), int(line[2], 16)))
        else:
            vals.append((int(line[0], 16), float(line[1])))
    return vals, rounds


def test_published_values_and_ties():
    vals, rounds = _rows()
    codes = np.array([c for c, _ in vals], dtype=np.uint8)
    got = oracle.e4m3_widen(codes)
    for (c, want), g in zip(vals, got):
        if math.isnan(want):
            assert math.isnan(g), hex(c)
        else:
            assert g == want and math.copysign(1.0, g) == math.copysign(1.0, want), hex(c)
    x = np.array([v for v, _ in rounds], dtype=np.float32)
    got = oracle.e4m3_round(x)
    assert [int(g) for g in got] == [c for _, c in rounds]


def test_widen_all_codes_against_torch():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    got = oracle.e4m3_widen(codes)
    nan = np.isnan(ref)
    assert list(np.nonzero(nan)[0]) == [0x7F, 0xFF]
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))


def test_round_against_torch_in_range():
    rng = np.random.default_rng(7)
    mag = np.exp2(rng.uniform(-12.0, math.log2(448.0), size=200_000)).astype(np.float32)
    x = (mag * rng.choice([-1.0, 1.0], size=mag.size)).astype(np.float32)
    # every midpoint between neighbouring values, and its fp32 neighbours on both sides
    grid = oracle.e4m3_widen(np.arange(0x7F, dtype=np.uint8))
    mid = ((grid[:-1] + grid[1:]) / 2).astype(np.float32)
    x = np.concatenate([x, mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(1e9)), -mid,
                        grid.astype(np.float32)])
    x = x[np.abs(x) <= 448.0]
    ref = torch.from_numpy(x.copy()).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle.e4m3_round(x)
    assert np.array_equal(got, ref)


def test_round_is_nearest_and_monotone():
    # brute force on a dense sweep: no other finite value is closer, and codes never decrease
    x = np.linspace(-460.0, 460.0, 40_001).astype(np.float32)
    got = oracle.e4m3_round(x)
    val = oracle.e4m3_widen(got)
    grid = oracle.e4m3_widen(np.arange(0x7F, dtype=np.uint8))
    grid = np.concatenate([-grid[::-1], grid])
    best = np.min(np.abs(x.astype(np.float64)[:, None] - grid[None, :]), axis=1)
    assert np.array_equal(np.abs(val - x.astype(np.float64)), best)
    assert np.all(np.diff(val) >= 0)


def test_quantize_multiplies_in_fp32_by_the_fp32_reciprocal():
    rng = np.random.default_rng(11)
    x = torch.from_numpy(rng.standard_normal(50_000).astype(np.float32)).to(torch.bfloat16)
    for scale in (1.0, 2.0 ** -6, 0.013, 3.7):
        inv = np.float32(1.0) / np.float32(scale)
        y = x.to(torch.float32).numpy() * inv                      # fp32 product
        want = torch.from_numpy(np.clip(y, -448.0, 448.0)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        got = oracle.e4m3_quantize(x, oracle.BF16, scale)
        assert np.array_equal(got, want)

def _rand_case(seed, L=37, Hq=4, Hkv=2, D=16):
    rng = np.random.default_rng(seed)
    q = torch.from_numpy(rng.standard_normal((1, Hq, D)).astype(np.float32)).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((L, Hkv, D)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((L, Hkv, D)).astype(np.float32)).to(torch.bfloat16)
    return q, k, v


def test_attention_over_codes_equals_attention_over_their_values():
    # with power-of-two scales the dequantised store is exact in fp32: the fp32 path of the
    # checker on those values is the same computation
    q, k, v = _rand_case(3)
    ks, vs = 2.0 ** -5, 2.0 ** -6
    kc, vc = oracle.e4m3_quantize(k, oracle.BF16, ks), oracle.e4m3_quantize(v, oracle.BF16, vs)
    out, lse, _ = oracle.decode_attention_e4m3(q, oracle.BF16, [kc], [vc], ks, vs, 4, 2, 16, want_lse=True)
    kd = (oracle.e4m3_widen(kc) * ks).astype(np.float32)
    vd = (oracle.e4m3_widen(vc) * vs).astype(np.float32)
    assert np.array_equal(kd.astype(np.float64), oracle.e4m3_widen(kc) * ks)
    ref, ref_lse, _ = oracle.decode_attention(q.to(torch.float32), [kd], [vd], 4, 2, 16, oracle.F32, want_lse=True)
    assert np.max(np.abs(out - ref)) < 1e-13
    assert np.max(np.abs(lse - ref_lse)) < 1e-13
    # and against torch's own dequantisation and softmax, in fp64
    kt = torch.from_numpy(kc.copy()).view(torch.float8_e4m3fn).to(torch.float64) * ks
    vt = torch.from_numpy(vc.copy()).view(torch.float8_e4m3fn).to(torch.float64) * vs
    qt = q.to(torch.float64)[0]
    for h in range(4):
        s = (kt[:, h // 2, :] @ qt[h]) / math.sqrt(16)
        o = torch.softmax(s, 0) @ vt[:, h // 2, :]
        assert torch.max(torch.abs(o - torch.from_numpy(out[0, h]))) < 1e-13
        assert abs(float(torch.logsumexp(s, 0)) - lse[0, h]) < 1e-13


def test_scales_enter_where_they_should():
    q, k, v = _rand_case(5)
    kc, vc = oracle.e4m3_quantize(k, oracle.BF16, 0.05), oracle.e4m3_quantize(v, oracle.BF16, 0.05)
    a, la, _ = oracle.decode_attention_e4m3(q, oracle.BF16, [kc], [vc], 0.05, 0.05, 4, 2, 16, want_lse=True)
    b, lb, _ = oracle.decode_attention_e4m3(q, oracle.BF16, [kc], [vc], 0.05, 0.1, 4, 2, 16, want_lse=True)
    # the value scale is linear in the output and absent from the scores
    assert np.allclose(b, a * (np.float64(np.float32(0.1)) / np.float64(np.float32(0.05))), rtol=1e-14, atol=0)
    assert np.array_equal(la, lb)
    # a key scale of zero flattens the softmax: the mean of the values, lse = log L
    c, lc, _ = oracle.decode_attention_e4m3(q, oracle.BF16, [kc], [vc], 0.0, 0.05, 4, 2, 16, want_lse=True)
    vm = (oracle.e4m3_widen(vc) * np.float64(np.float32(0.05))).mean(axis=0)
    for h in range(4):
        assert np.allclose(c[0, h], vm[h // 2], rtol=1e-13, atol=1e-15)
    assert np.allclose(lc, math.log(37), rtol=1e-14)


def test_store_quantises_at_append():
    q, k, v = _rand_case(9)
    st = oracle.KVStore(2, 2, 16, oracle.BF16, kv_e4m3=True, k_scale=[1.0, 0.03], v_scale=[1.0, 0.02])
    st.append(7, 1, k[:30], v[:30])
    st.append(7, 1, k[30:], v[30:])
    kk, vv = st.gathered(7, 1)
    assert kk.dtype == np.uint8 and kk.shape == (37, 2, 16)
    assert np.array_equal(kk, oracle.e4m3_quantize(k, oracle.BF16, 0.03))
    out, _, _ = st.decode_attention(1, [7], q, 4)
    ref, _, _ = oracle.decode_attention_e4m3(q, oracle.BF16, [kk], [vv], 0.03, 0.02, 4, 2, 16)
    assert np.array_equal(out, ref)
