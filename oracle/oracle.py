"""ctypes face of the CPU checker (oracle/odma_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The GPU library never imports it and shares no
code with it.  Everything numerical happens in the C file; this module moves
arrays in and out and keeps the checker's own per-request K/V store (rows in
the order they were appended, token-major), which is independent of the device
pool layout.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "odma_oracle.c")
_LIB = os.path.join(_HERE, "libodma_oracle.so")

F32, BF16, E4M3 = 0, 1, 2

OK, ERR_INVALID, ERR_NOMEM, ERR_UNKNOWN_REQ, ERR_DUP_REQ, ERR_OVERFLOW = range(6)


def build(force: bool = False) -> str:
    """Compile the checker with gcc (plain C99 + OpenMP) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i32p, i64p, u64p, dp = (C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                C.POINTER(C.c_uint64), C.POINTER(C.c_double))
        L.oracle_decode_attention.restype = C.c_int
        L.oracle_decode_attention.argtypes = [C.c_int, C.c_void_p, C.POINTER(C.c_void_p),
                                              C.POINTER(C.c_void_p), i32p, C.c_int, C.c_int,
                                              C.c_int, C.c_int, dp, dp, C.c_int]
        L.oracle_attention_weights.restype = C.c_double
        L.oracle_attention_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                               C.c_int, C.c_int, C.c_int, C.c_int, dp, dp]
        L.oracle_attention_chunked.restype = None
        L.oracle_attention_chunked.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                               C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, dp]
        L.oracle_decode_attention_e4m3.restype = C.c_int
        L.oracle_decode_attention_e4m3.argtypes = [C.c_int, C.c_void_p, C.c_int, C.POINTER(C.c_void_p),
                                                   C.POINTER(C.c_void_p), C.c_float, C.c_float, i32p, C.c_int,
                                                   C.c_int, C.c_int, dp, dp, C.c_int]
        L.oracle_e4m3_widen.restype = None
        L.oracle_e4m3_widen.argtypes = [C.c_void_p, C.c_size_t, dp]
        L.oracle_e4m3_round.restype = None
        L.oracle_e4m3_round.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        L.oracle_e4m3_quantize.restype = None
        L.oracle_e4m3_quantize.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_float, C.c_void_p]
        L.ora_create.restype = C.c_void_p
        L.ora_create.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64,
                                 C.c_int64, C.c_int64, C.c_int64, C.c_int, i32p, C.c_int32, C.c_int,
                                 C.c_int, C.c_int, C.c_int]
        L.ora_destroy.argtypes = [C.c_void_p]
        L.ora_geometry.argtypes = [C.c_void_p, i64p]
        L.ora_set_buckets.argtypes = [C.c_void_p, i32p, C.c_int]
        L.ora_get_buckets.argtypes = [C.c_void_p, i32p, u64p]
        L.ora_reserve.argtypes = [C.c_void_p, C.c_uint64, C.c_int64, i64p]
        L.ora_reserve_uncertain.argtypes = [C.c_void_p, C.c_uint64, C.c_int64, C.c_int64, i64p]
        L.ora_ensure.argtypes = [C.c_void_p, C.c_uint64, C.c_int64, i64p, i32p]
        L.ora_add_len.argtypes = [C.c_void_p, C.c_uint64, C.c_int64]
        L.ora_get_len.restype = C.c_int64
        L.ora_get_len.argtypes = [C.c_void_p, C.c_uint64]
        L.ora_release.argtypes = [C.c_void_p, C.c_uint64]
        L.ora_stats.argtypes = [C.c_void_p, i64p]
        L.ora_owner_array.restype = C.POINTER(C.c_int32)
        L.ora_owner_array.argtypes = [C.c_void_p]
        L.ora_live.restype = C.c_int64
        L.ora_live.argtypes = [C.c_void_p, C.c_int64, u64p, i64p, i64p, i64p, i32p]
        _lib = L
    return _lib


# ---------------------------------------------------------------------------
# attention
# ---------------------------------------------------------------------------


def _as_store(x, dtype_code: int) -> np.ndarray:
    """Accept a torch tensor (fp32 / bf16) or numpy array; return the raw storage array."""
    if hasattr(x, "detach"):
        import torch
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16)
        return x.numpy()
    return np.ascontiguousarray(x)


def dtype_code(torch_dtype) -> int:
    import torch
    if torch_dtype == torch.float32:
        return F32
    if torch_dtype == torch.bfloat16:
        return BF16
    raise ValueError(f"unsupported dtype {torch_dtype}")


def decode_attention(q, K: Sequence, V: Sequence, q_heads: int, kv_heads: int, head_dim: int,
                     dtype: int, threads: int = 0, want_lse: bool = False):
    """Dense fp64 attention for a batch.

    q: [n, Hq, D]; K[i], V[i]: [L_i, Hkv, D] (torch fp32/bf16 tensors, or raw numpy
    float32 / uint16 arrays).  Returns (out [n, Hq, D] float64, lse or None, threads used).
    """
    L = lib()
    qa = _as_store(q, dtype)
    n = qa.shape[0]
    Ks = [_as_store(k, dtype) for k in K]
    Vs = [_as_store(v, dtype) for v in V]
    lens = np.array([k.shape[0] for k in Ks], dtype=np.int32)
    kp = (C.c_void_p * n)(*[k.ctypes.data for k in Ks])
    vp = (C.c_void_p * n)(*[v.ctypes.data for v in Vs])
    out = np.empty((n, q_heads, head_dim), dtype=np.float64)
    lse = np.empty((n, q_heads), dtype=np.float64) if want_lse else None
    used = L.oracle_decode_attention(
        n, qa.ctypes.data, kp, vp, lens.ctypes.data_as(C.POINTER(C.c_int32)), q_heads, kv_heads,
        head_dim, dtype, out.ctypes.data_as(C.POINTER(C.c_double)),
        lse.ctypes.data_as(C.POINTER(C.c_double)) if want_lse else None, threads)
    return out, lse, used


def e4m3_widen(codes) -> np.ndarray:
    """The values (float64) of an array of E4M3 codes (uint8)."""
    c = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(c.shape, dtype=np.float64)
    lib().oracle_e4m3_widen(c.ctypes.data, c.size, out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


def e4m3_round(x) -> np.ndarray:
    """Nearest E4M3 code (ties to even, saturating at +-448) of each float32."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint8)
    lib().oracle_e4m3_round(a.ctypes.data, a.size, out.ctypes.data)
    return out


def inv_scale(scale: float) -> np.float32:
    """The fp32 reciprocal an append multiplies by: 1 / scale, both in fp32, correctly rounded."""
    return np.float32(1.0) / np.float32(scale)


def e4m3_quantize(x, dtype: int, scale: float) -> np.ndarray:
    """Codes an append of `x` (fp32 / bf16 rows) stores in an E4M3 slab with dequantisation scale `scale`."""
    a = _as_store(x, dtype)
    out = np.empty(a.shape, dtype=np.uint8)
    lib().oracle_e4m3_quantize(a.ctypes.data, dtype, a.size, C.c_float(float(inv_scale(scale))), out.ctypes.data)
    return out


def decode_attention_e4m3(q, qdtype: int, K: Sequence, V: Sequence, k_scale: float, v_scale: float,
                          q_heads: int, kv_heads: int, head_dim: int, threads: int = 0, want_lse: bool = False):
    """Dense fp64 attention with K[i], V[i] as E4M3 code arrays [L_i, Hkv, D] (uint8) and their scales."""
    L = lib()
    qa = _as_store(q, qdtype)
    n = qa.shape[0]
    Ks = [np.ascontiguousarray(k, dtype=np.uint8) for k in K]
    Vs = [np.ascontiguousarray(v, dtype=np.uint8) for v in V]
    lens = np.array([k.shape[0] for k in Ks], dtype=np.int32)
    kp = (C.c_void_p * n)(*[k.ctypes.data for k in Ks])
    vp = (C.c_void_p * n)(*[v.ctypes.data for v in Vs])
    out = np.empty((n, q_heads, head_dim), dtype=np.float64)
    lse = np.empty((n, q_heads), dtype=np.float64) if want_lse else None
    used = L.oracle_decode_attention_e4m3(
        n, qa.ctypes.data, qdtype, kp, vp, C.c_float(float(np.float32(k_scale))), C.c_float(float(np.float32(v_scale))),
        lens.ctypes.data_as(C.POINTER(C.c_int32)), q_heads, kv_heads, head_dim,
        out.ctypes.data_as(C.POINTER(C.c_double)), lse.ctypes.data_as(C.POINTER(C.c_double)) if want_lse else None,
        threads)
    return out, lse, used


def attention_weights(q, K, V, h: int, q_heads: int, kv_heads: int, head_dim: int, dtype: int):
    """(out [D], weights [L], lse) of one request and one query head."""
    L = lib()
    qa, ka, va = _as_store(q, dtype), _as_store(K, dtype), _as_store(V, dtype)
    n_keys = ka.shape[0]
    out = np.empty(head_dim, dtype=np.float64)
    w = np.empty(n_keys, dtype=np.float64)
    lse = L.oracle_attention_weights(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, n_keys, h,
                                     q_heads, kv_heads, head_dim, dtype,
                                     out.ctypes.data_as(C.POINTER(C.c_double)),
                                     w.ctypes.data_as(C.POINTER(C.c_double)))
    return out, w, lse


def attention_chunked(q, K, V, h: int, q_heads: int, kv_heads: int, head_dim: int, dtype: int,
                      chunk: int) -> np.ndarray:
    L = lib()
    qa, ka, va = _as_store(q, dtype), _as_store(K, dtype), _as_store(V, dtype)
    out = np.empty(head_dim, dtype=np.float64)
    L.oracle_attention_chunked(qa.ctypes.data, ka.ctypes.data, va.ctypes.data, ka.shape[0], h,
                               q_heads, kv_heads, head_dim, dtype, chunk,
                               out.ctypes.data_as(C.POINTER(C.c_double)))
    return out


class KVStore:
    """The checker's own KV cache: per (request, layer) the rows appended so far, in order."""

    def __init__(self, layers: int, kv_heads: int, head_dim: int, dtype: int, kv_e4m3: bool = False,
                 k_scale: Optional[Sequence[float]] = None, v_scale: Optional[Sequence[float]] = None):
        """`dtype`: the type of q and of the rows given to append.  With `kv_e4m3` the store holds
        E4M3 codes, quantised at append with the layer's scale (k_scale[l], v_scale[l]; default 1)."""
        self.layers, self.kv_heads, self.head_dim, self.dtype = layers, kv_heads, head_dim, dtype
        self.kv_e4m3 = kv_e4m3
        self.k_scale = [float(x) for x in (k_scale if k_scale is not None else [1.0] * layers)]
        self.v_scale = [float(x) for x in (v_scale if v_scale is not None else [1.0] * layers)]
        self.k: Dict[Tuple[int, int], List[np.ndarray]] = {}
        self.v: Dict[Tuple[int, int], List[np.ndarray]] = {}

    def append(self, req: int, layer: int, k_rows, v_rows) -> None:
        """k_rows, v_rows: [n_tok, Hkv, D]."""
        if self.kv_e4m3:
            self.k.setdefault((req, layer), []).append(e4m3_quantize(k_rows, self.dtype, self.k_scale[layer]))
            self.v.setdefault((req, layer), []).append(e4m3_quantize(v_rows, self.dtype, self.v_scale[layer]))
            return
        self.k.setdefault((req, layer), []).append(_as_store(k_rows, self.dtype).copy())
        self.v.setdefault((req, layer), []).append(_as_store(v_rows, self.dtype).copy())

    def gathered(self, req: int, layer: int) -> Tuple[np.ndarray, np.ndarray]:
        k = np.concatenate(self.k[(req, layer)], axis=0)
        v = np.concatenate(self.v[(req, layer)], axis=0)
        self.k[(req, layer)], self.v[(req, layer)] = [k], [v]
        return k, v

    def length(self, req: int, layer: int = 0) -> int:
        return sum(x.shape[0] for x in self.k.get((req, layer), []))

    def drop(self, req: int) -> None:
        for l in range(self.layers):
            self.k.pop((req, l), None)
            self.v.pop((req, l), None)

    def decode_attention(self, layer: int, reqs: Sequence[int], q, q_heads: int, threads: int = 0,
                         want_lse: bool = False):
        Ks, Vs = zip(*[self.gathered(r, layer) for r in reqs])
        if self.kv_e4m3:
            return decode_attention_e4m3(q, self.dtype, Ks, Vs, self.k_scale[layer], self.v_scale[layer], q_heads,
                                         self.kv_heads, self.head_dim, threads, want_lse)
        return decode_attention(q, Ks, Vs, q_heads, self.kv_heads, self.head_dim, self.dtype,
                                threads, want_lse)


def prefill_attention(store: "KVStore", layer: int, reqs: Sequence[int], n_new: Sequence[int], q, q_heads: int,
                      threads: int = 0):
    """Causal attention of a prefill chunk, by its definition: the store already holds the chunk;
    new token j of request i (its n_new[i] last tokens) attends keys [0, its own position].  q:
    [sum(n_new), Hq, D], tokens in request order then position order.  Each token is one dense
    fp64 attention over a prefix of the request's rows.  Returns (out [sum(n_new), Hq, D], lse)."""
    Ks, Vs = [], []
    for r, k in zip(reqs, n_new):
        K, V = store.gathered(r, layer)
        L = K.shape[0]
        for j in range(k):
            Ks.append(K[: L - k + j + 1])
            Vs.append(V[: L - k + j + 1])
    if store.kv_e4m3:
        out, lse, _ = decode_attention_e4m3(q, store.dtype, Ks, Vs, store.k_scale[layer], store.v_scale[layer], q_heads,
                                            store.kv_heads, store.head_dim, threads, True)
    else:
        out, lse, _ = decode_attention(q, Ks, Vs, q_heads, store.kv_heads, store.head_dim, store.dtype, threads, True)
    return out, lse


# ---------------------------------------------------------------------------
# allocator
# ---------------------------------------------------------------------------

Slab = Tuple[int, int, int, int, int]   # base_tok, cap_tok, pool_id, bucket_id, epoch


class Allocator:
    """Brute-force bucket allocator (owner array per token)."""

    def __init__(self, pool_bytes: int, layers: int, kv_heads: int, head_dim: int, elem_bytes: int,
                 safety_pct: int = 10, max_len: int = 32768, granule: int = 16, window: int = 10000,
                 refresh: int = 1000, p_num: Sequence[int] = (1, 2, 3, 4), p_den: int = 4,
                 gamma_permille: int = 200, tau_permille: int = 800, growth: int = 2,
                 large_fixed: int = 0):
        self._L = lib()
        pn = (C.c_int32 * len(p_num))(*p_num)
        self._h = self._L.ora_create(pool_bytes, layers, kv_heads, head_dim, elem_bytes, safety_pct,
                                     max_len, granule, window, refresh, len(p_num), pn, p_den,
                                     gamma_permille, tau_permille, growth, large_fixed)
        if not self._h:
            raise ValueError("invalid allocator configuration")
        g = (C.c_int64 * 3)()
        self._L.ora_geometry(self._h, g)
        self.T, self.S, self.M = int(g[0]), int(g[1]), int(g[2])
        self.granule = granule

    def __del__(self):
        if getattr(self, "_h", None):
            self._L.ora_destroy(self._h)
            self._h = None

    def set_buckets(self, b: Sequence[int]) -> int:
        arr = (C.c_int32 * len(b))(*b)
        return self._L.ora_set_buckets(self._h, arr, len(b))

    def get_buckets(self) -> Tuple[Tuple[int, ...], int]:
        arr = (C.c_int32 * 8)()
        ep = C.c_uint64()
        n = self._L.ora_get_buckets(self._h, arr, C.byref(ep))
        return tuple(arr[i] for i in range(n)), int(ep.value)

    def reserve(self, req: int, predicted: int) -> Tuple[int, Optional[Slab]]:
        out = (C.c_int64 * 5)()
        rc = self._L.ora_reserve(self._h, req, predicted, out)
        return rc, (tuple(int(x) for x in out) if rc == OK else None)

    def reserve_uncertain(self, req: int, l_hat: int, u_permille: int):
        out = (C.c_int64 * 5)()
        rc = self._L.ora_reserve_uncertain(self._h, req, l_hat, u_permille, out)
        return rc, (tuple(int(x) for x in out) if rc == OK else None)

    def ensure_capacity(self, req: int, need: int):
        out = (C.c_int64 * 5)()
        mig = C.c_int32()
        rc = self._L.ora_ensure(self._h, req, need, out, C.byref(mig))
        return rc, (tuple(int(x) for x in out) if rc == OK else None), int(mig.value)

    def add_len(self, req: int, n_new: int) -> int:
        return self._L.ora_add_len(self._h, req, n_new)

    def get_len(self, req: int) -> int:
        return int(self._L.ora_get_len(self._h, req))

    def release(self, req: int) -> int:
        return self._L.ora_release(self._h, req)

    def stats(self) -> Dict[str, int]:
        out = (C.c_int64 * 12)()
        self._L.ora_stats(self._h, out)
        keys = ["live", "reserved_live", "used_live", "completed", "sum_len_completed",
                "sum_cap_completed", "migrations", "nomem", "routed_large", "safety_live",
                "safety_peak", "observed"]
        return {k: int(out[i]) for i, k in enumerate(keys)}

    def owner_array(self) -> np.ndarray:
        p = self._L.ora_owner_array(self._h)
        return np.ctypeslib.as_array(p, shape=(self.T,)).copy()

    def live(self, n_max: int = 1 << 16):
        ids = (C.c_uint64 * n_max)()
        base = (C.c_int64 * n_max)()
        cap = (C.c_int64 * n_max)()
        ln = (C.c_int64 * n_max)()
        pool = (C.c_int32 * n_max)()
        k = self._L.ora_live(self._h, n_max, ids, base, cap, ln, pool)
        return [(int(ids[i]), int(base[i]), int(cap[i]), int(ln[i]), int(pool[i])) for i in range(k)]

    # adapter used by workloads.run_closed_loop -----------------------------------------------
    def alloc(self, req, predicted):
        rc, slab = self.reserve(req, predicted)
        return slab[:4] if rc == OK else None

    def ensure(self, req, need):
        rc, slab, mig = self.ensure_capacity(req, need)
        if rc == ERR_NOMEM:
            return None
        if rc != OK:
            raise RuntimeError(f"oracle ensure_capacity({req},{need}) -> {rc}")
        return slab[:4], mig

    def commit(self, reqs, n_new):
        for r in reqs:
            rc = self.add_len(r, n_new)
            assert rc == OK, (r, n_new, rc)

    def free(self, req):
        rc = self.release(req)
        assert rc == OK

    def buckets(self):
        return self.get_buckets()
