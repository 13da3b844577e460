"""Thin ctypes binding of libodma.so: same names as the C ABI, argument marshalling only.

Every computation happens inside the shared library (CUDA kernels and the C++ host
allocator).  Importing this module loads the library and raises ImportError when it has
not been built (`python -m paper_2512_09427_b200.build`); there is no fallback path.
Device buffers are passed as integers (`tensor.data_ptr()`), streams as the integer
`torch.cuda.current_stream().cuda_stream`.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libodma.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_09427_b200.build`")
_lib = C.CDLL(LIB_PATH)

MAX_BUCKETS = 8
OK, ERR_INVALID, ERR_NOMEM, ERR_UNKNOWN_REQ, ERR_DUP_REQ, ERR_OVERFLOW, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = range(9)
DTYPE_F32, DTYPE_BF16, DTYPE_FP8_E4M3 = 0, 1, 2
DECODE_AUTO, DECODE_TCGEN05, DECODE_MMA_SYNC = 0, 1, 2
READOUT_AUTO, READOUT_LATE, READOUT_AT_ONCE = 0, 1, 2
K_APPEND, K_DECODE, K_COMBINE, K_MIGRATE, K_PROBE = range(5)


class Config(C.Structure):
    _fields_ = [("safety_pct", C.c_int32), ("max_len", C.c_int32), ("granule", C.c_int32),
                ("window", C.c_int32), ("refresh", C.c_int32), ("n_levels", C.c_int32),
                ("p_num", C.c_int32 * MAX_BUCKETS), ("p_den", C.c_int32),
                ("gamma_permille", C.c_int32), ("tau_permille", C.c_int32), ("growth", C.c_int32),
                ("large_fixed", C.c_int32), ("max_batch", C.c_int32), ("max_group", C.c_int32),
                ("plan_ctas", C.c_int32), ("fused_combine", C.c_int32), ("fused_append", C.c_int32),
                ("decode_kernel", C.c_int32), ("chain_launches", C.c_int32), ("span_layers", C.c_int32), ("async_recal", C.c_int32), ("cluster_observe", C.c_int32), ("readout", C.c_int32)]


class Slab(C.Structure):
    _fields_ = [("base_tok", C.c_int32), ("cap_tok", C.c_int32), ("pool_id", C.c_int32),
                ("bucket_id", C.c_int32), ("epoch", C.c_uint64)]

    def astuple(self) -> Tuple[int, int, int, int, int]:
        return (self.base_tok, self.cap_tok, self.pool_id, self.bucket_id, self.epoch)


class Stats(C.Structure):
    _fields_ = [(k, C.c_int64) for k in
                ("total_tokens", "safety_tokens", "main_tokens", "live", "reserved_live", "used_live",
                 "completed", "sum_len_completed", "sum_cap_completed", "migrations", "nomem",
                 "routed_large", "safety_live", "safety_peak", "observed")] + [("epoch", C.c_uint64)]

    def asdict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class Tables(C.Structure):
    _fields_ = [("d_table", C.c_void_p)] + [(k, C.c_int32) for k in
                ("n", "n_new_total", "n_items", "n_ctas", "n_combine", "words", "off_base", "off_cap",
                 "off_len", "off_cu_new", "off_cta", "off_items", "off_combine", "tile_tokens", "one_new_each",
                 "reserved")] + \
               [("kv_tokens", C.c_int64), ("epoch", C.c_uint64)]


class SimRequest(C.Structure):
    _fields_ = [("arrival_ns", C.c_int64), ("prompt", C.c_int32), ("total", C.c_int32), ("predicted", C.c_int32),
                ("u_permille", C.c_int32)]


class SimParams(C.Structure):
    _fields_ = [("policy", C.c_int32), ("max_batch", C.c_int32), ("layers", C.c_int32), ("reserved", C.c_int32),
                ("base_ns", C.c_int64), ("ps_per_token", C.c_int64)]


class SimResult(C.Structure):
    _fields_ = [(k, C.c_int64) for k in
                ("completed", "failed", "tokens_out", "tokens_lost", "steps", "makespan_ns", "sum_actual", "sum_reserved",
                 "conc_time", "reserved_time", "used_time", "migrations", "preemptions", "stalls", "deferred")]

    def asdict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


SIM_STATIC, SIM_PAGED16, SIM_ODMA = 0, 1, 2

_vp, _i32, _u64, _i64 = C.c_void_p, C.c_int32, C.c_uint64, C.c_int64
_i32p, _u64p = C.POINTER(C.c_int32), C.POINTER(C.c_uint64)

_SIGS = {
    "odma_config_default": (None, [C.POINTER(Config)]),
    "odma_strerror": (C.c_char_p, [_i32]),
    "odma_pool_create": (_i32, [_vp, _u64, _i32, _i32, _i32, _i32, C.POINTER(Config), C.POINTER(_vp)]),
    "odma_pool_destroy": (_i32, [_vp]),
    "odma_recal_flush": (_i32, [_vp]),
    "odma_drain_observations": (_i32, [_vp, _i32p, _i32, _i32p]),
    "odma_observe": (_i32, [_vp, _i32p, _i32]),
    "odma_set_kv_scales": (_i32, [_vp, C.POINTER(C.c_float), C.POINTER(C.c_float)]),
    "odma_set_buckets": (_i32, [_vp, _i32p, _i32]),
    "odma_get_buckets": (_i32, [_vp, _i32p, _i32p, _u64p]),
    "odma_alloc": (_i32, [_vp, _u64, _i32, C.POINTER(Slab)]),
    "odma_alloc_uncertain": (_i32, [_vp, _u64, _i32, _i32, C.POINTER(Slab)]),
    "odma_ensure_capacity": (_i32, [_vp, _u64, _i32, _vp, C.POINTER(Slab), _i32p]),
    "odma_free": (_i32, [_vp, _u64]),
    "odma_commit_step": (_i32, [_vp, _u64p, _i32, _i32p]),
    "odma_get_slab": (_i32, [_vp, _u64, C.POINTER(Slab), _i32p]),
    "odma_get_stats": (_i32, [_vp, C.POINTER(Stats)]),
    "odma_tables_bytes": (_u64, [_vp, _i32]),
    "odma_plan_host": (_i32, [_vp, _u64p, _i32p, _i32, _i32p, _u64, C.POINTER(Tables)]),
    "odma_build_tables": (_i32, [_vp, _u64p, _i32p, _i32, _vp, _u64, _vp, C.POINTER(Tables)]),
    "odma_build_prefill_tables": (_i32, [_vp, _u64p, _i32p, _i32, _vp, _u64, _vp, C.POINTER(Tables)]),
    "odma_append_kv": (_i32, [_vp, _i32, C.POINTER(Tables), _vp, _vp, _vp]),
    "odma_decode_attention": (_i32, [_vp, _i32, _vp, _i32, C.POINTER(Tables), _vp, _vp, _vp]),
    "odma_decode_step_host": (_i32, [_vp, _i32, _i32, _u64p, _i32, _vp, _vp, _vp, _vp, _vp]),
    "odma_decode_step": (_i32, [_vp, _i32, _i32, _i32, _u64p, _i32, _vp, _vp, _vp, _vp, _vp, _vp,
                                C.POINTER(Tables)]),
    "odma_decode_attention_static": (_i32, [_vp, _vp, _i32, _vp, _i32, C.POINTER(Tables), _vp, _vp, _vp]),
    "odma_check_status": (_i32, [_vp, _vp]),
    "odma_selftest_timeout": (_i32, [_vp, _i32, _vp]),
    "odma_read_probe": (_i32, [_vp, _i32, _i32, C.POINTER(Tables), _vp]),
    "odma_profile_enable": (_i32, [_vp, _i32]),
    "odma_profile_read": (_i32, [_vp, _i32, C.POINTER(C.c_double), C.POINTER(_i64)]),
    "odma_sim_run": (_i32, [_vp, C.POINTER(SimParams), C.POINTER(SimRequest), _i32, C.POINTER(SimResult)]),
    "odma_paged_create": (_i32, [_vp, _vp, _u64, C.POINTER(_vp)]),
    "odma_paged_destroy": (_i32, [_vp]),
    "odma_paged_build": (_i32, [_vp, C.POINTER(Tables), _i32p, _u64, _vp, _i32, _vp]),
    "odma_decode_attention_paged": (_i32, [_vp, _i32, _vp, _i32, C.POINTER(Tables), _vp, _i32, _vp, _vp, _vp]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)
    _fn.restype, _fn.argtypes = _res, _args

EXPORTS = tuple(_SIGS)


class OdmaError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


def strerror(code: int) -> str:
    return _lib.odma_strerror(code).decode()


def config_default() -> Config:
    cfg = Config()
    _lib.odma_config_default(C.byref(cfg))
    return cfg


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise OdmaError(rc, what)


def _u64arr(xs: Sequence[int]):
    return (C.c_uint64 * len(xs))(*xs)


def _i32arr(xs: Optional[Sequence[int]]):
    return None if xs is None else (C.c_int32 * len(xs))(*[int(x) for x in xs])


class Pool:
    """Handle of one odma_pool.  Methods mirror the C entry points one to one; those that can
    fail in normal operation (alloc, ensure_capacity) return the status code, the rest raise."""

    def __init__(self, dev_base: int, nbytes: int, layers: int, kv_heads: int, head_dim: int,
                 dtype: int, cfg: Optional[Config] = None):
        self._h = C.c_void_p()
        self.layers, self.kv_heads, self.head_dim, self.dtype = layers, kv_heads, head_dim, dtype
        _check(_lib.odma_pool_create(dev_base or None, nbytes, layers, kv_heads, head_dim, dtype,
                                     C.byref(cfg) if cfg is not None else None, C.byref(self._h)),
               "odma_pool_create")

    def destroy(self) -> None:
        if self._h:
            _lib.odma_pool_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def recal_flush(self) -> None:
        _check(_lib.odma_recal_flush(self._h), "odma_recal_flush")

    def drain_observations(self, cap: int = 1 << 20) -> list:
        """Lengths of the requests completed here since the last drain (oldest first)."""
        buf = (C.c_int32 * cap)()
        n = C.c_int32()
        _check(_lib.odma_drain_observations(self._h, buf, cap, C.byref(n)), "odma_drain_observations")
        return list(buf[: n.value])

    def observe(self, lengths: Sequence[int]) -> None:
        _check(_lib.odma_observe(self._h, _i32arr(list(lengths)), len(lengths)), "odma_observe")

    def set_kv_scales(self, k_scale: Sequence[float], v_scale: Sequence[float]) -> None:
        """Per-layer dequantisation scales of an 8-bit (E4M3) pool."""
        assert len(k_scale) == self.layers and len(v_scale) == self.layers
        _check(_lib.odma_set_kv_scales(self._h, (C.c_float * self.layers)(*k_scale), (C.c_float * self.layers)(*v_scale)),
               "odma_set_kv_scales")

    # -- boundaries --------------------------------------------------------------------------
    def set_buckets(self, b: Sequence[int]) -> int:
        return _lib.odma_set_buckets(self._h, _i32arr(b), len(b))

    def get_buckets(self) -> Tuple[Tuple[int, ...], int]:
        arr = (C.c_int32 * MAX_BUCKETS)()
        n, ep = C.c_int32(), C.c_uint64()
        _check(_lib.odma_get_buckets(self._h, arr, C.byref(n), C.byref(ep)), "odma_get_buckets")
        return tuple(arr[i] for i in range(n.value)), int(ep.value)

    # -- reserve / release -------------------------------------------------------------------
    def alloc(self, req: int, predicted_len: int) -> Tuple[int, Optional[Tuple[int, ...]]]:
        s = Slab()
        rc = _lib.odma_alloc(self._h, req, predicted_len, C.byref(s))
        return rc, (s.astuple() if rc == OK else None)

    def alloc_uncertain(self, req: int, l_hat: int, u_permille: int):
        s = Slab()
        rc = _lib.odma_alloc_uncertain(self._h, req, l_hat, u_permille, C.byref(s))
        return rc, (s.astuple() if rc == OK else None)

    def ensure_capacity(self, req: int, needed_len: int, stream: int = 0):
        s, mig = Slab(), C.c_int32()
        rc = _lib.odma_ensure_capacity(self._h, req, needed_len, stream or None, C.byref(s), C.byref(mig))
        return rc, (s.astuple() if rc == OK else None), int(mig.value)

    def free(self, req: int) -> int:
        return _lib.odma_free(self._h, req)

    def commit_step(self, reqs, n_new: Optional[Sequence[int]] = None) -> int:
        arr = reqs if isinstance(reqs, C.Array) else _u64arr(reqs)
        return _lib.odma_commit_step(self._h, arr, len(arr), _i32arr(n_new))

    def get_slab(self, req: int):
        s, ln = Slab(), C.c_int32()
        rc = _lib.odma_get_slab(self._h, req, C.byref(s), C.byref(ln))
        return rc, (s.astuple() if rc == OK else None), int(ln.value)

    def get_stats(self) -> dict:
        st = Stats()
        _check(_lib.odma_get_stats(self._h, C.byref(st)), "odma_get_stats")
        return st.asdict()

    # -- per-step tables ---------------------------------------------------------------------
    def tables_bytes(self, n: int) -> int:
        return int(_lib.odma_tables_bytes(self._h, n))

    def plan_host(self, reqs: Sequence[int], n_new: Optional[Sequence[int]] = None):
        """Returns (status, Tables, list of int32 words) without touching the device."""
        n = len(reqs)
        nbytes = self.tables_bytes(n)
        buf = (C.c_int32 * (nbytes // 4))()
        t = Tables()
        rc = _lib.odma_plan_host(self._h, _u64arr(reqs), _i32arr(n_new), n, buf, nbytes, C.byref(t))
        return rc, t, (list(buf[:t.words]) if rc == OK else None)

    def build_tables(self, reqs: Sequence[int], d_table: int, table_bytes: int, stream: int = 0,
                     n_new: Optional[Sequence[int]] = None) -> Tables:
        t = Tables()
        _check(_lib.odma_build_tables(self._h, _u64arr(reqs), _i32arr(n_new), len(reqs), d_table,
                                      table_bytes, stream or None, C.byref(t)), "odma_build_tables")
        return t

    def build_prefill_tables(self, reqs: Sequence[int], n_new: Sequence[int], d_table: int, table_bytes: int,
                             stream: int = 0) -> Tables:
        """Plan of the causal attention of a prefill chunk: one stream per new token."""
        t = Tables()
        _check(_lib.odma_build_prefill_tables(self._h, _u64arr(reqs), _i32arr(n_new), len(reqs), d_table,
                                              table_bytes, stream or None, C.byref(t)), "odma_build_prefill_tables")
        return t

    # -- kernels -----------------------------------------------------------------------------
    def append_kv(self, layer: int, tables: Tables, k_new: int, v_new: int, stream: int = 0) -> None:
        _check(_lib.odma_append_kv(self._h, layer, C.byref(tables), k_new, v_new, stream or None),
               "odma_append_kv")

    def decode_attention(self, layer: int, q: int, q_heads: int, tables: Tables, out: int,
                         lse: int = 0, stream: int = 0) -> None:
        _check(_lib.odma_decode_attention(self._h, layer, q, q_heads, C.byref(tables), out,
                                          lse or None, stream or None), "odma_decode_attention")

    def decode_step_host(self, layer: int, q_heads: int, reqs, h_q: int, h_k_new: int, h_v_new: int,
                         h_out: int, stream: int = 0) -> None:
        arr = reqs if isinstance(reqs, C.Array) else _u64arr(reqs)
        _check(_lib.odma_decode_step_host(self._h, layer, q_heads, arr, len(arr), h_q, h_k_new, h_v_new,
                                          h_out, stream or None), "odma_decode_step_host")

    def decode_step(self, layer: int, n_layers: int, q_heads: int, reqs, d_q: int, d_k_new: int,
                    d_v_new: int, d_out: int, lse: int = 0, stream: int = 0,
                    tables: Optional[Tables] = None) -> None:
        arr = reqs if isinstance(reqs, C.Array) else _u64arr(reqs)
        _check(_lib.odma_decode_step(self._h, layer, n_layers, q_heads, arr, len(arr), d_q, d_k_new,
                                     d_v_new, d_out, lse or None, stream or None,
                                     C.byref(tables) if tables is not None else None), "odma_decode_step")

    def decode_attention_static(self, dev_base: int, layer: int, q: int, q_heads: int, tables: Tables,
                                out: int, lse: int = 0, stream: int = 0) -> int:
        """odma_decode_attention_static: same result as decode_attention, no device allocation
        anywhere on the call (split partials live in a fixed array inside the library).
        Returns the status code (ERR_TOO_LARGE beyond the array's limits)."""
        return _lib.odma_decode_attention_static(self._h, dev_base, layer, q, q_heads, C.byref(tables),
                                                 out, lse or None, stream or None)

    def check_status(self, stream: int = 0) -> int:
        return _lib.odma_check_status(self._h, stream or None)

    def selftest_timeout(self, limit_ms: int, stream: int = 0) -> int:
        return _lib.odma_selftest_timeout(self._h, limit_ms, stream or None)

    def sim_run(self, policy: int, requests, max_batch: int, layers: int, base_ns: int, ps_per_token: int) -> dict:
        """requests: sequence of (arrival_ns, prompt, total, predicted, u_permille)."""
        arr = (SimRequest * len(requests))(*[SimRequest(*[int(x) for x in r]) for r in requests])
        prm = SimParams(policy, max_batch, layers, 0, base_ns, ps_per_token)
        res = SimResult()
        _check(_lib.odma_sim_run(self._h, C.byref(prm), arr, len(requests), C.byref(res)), "odma_sim_run")
        return res.asdict()

    def read_probe(self, layer: int, q_heads: int, tables: Tables, stream: int = 0) -> None:
        _check(_lib.odma_read_probe(self._h, layer, q_heads, C.byref(tables), stream or None),
               "odma_read_probe")

    def profile_enable(self, on: bool) -> None:
        _check(_lib.odma_profile_enable(self._h, int(on)), "odma_profile_enable")

    def profile_read(self, kernel: int) -> Tuple[float, int]:
        ms, cnt = C.c_double(), C.c_int64()
        _check(_lib.odma_profile_read(self._h, kernel, C.byref(ms), C.byref(cnt)), "odma_profile_read")
        return float(ms.value), int(cnt.value)


class Paged:
    """Handle of one odma_paged (page-16 copy of a pool, for the contiguity ablation)."""

    def __init__(self, pool: Pool, d_pages: int, nbytes: int):
        self._h = C.c_void_p()
        self.pool = pool
        _check(_lib.odma_paged_create(pool._h, d_pages, nbytes, C.byref(self._h)), "odma_paged_create")

    def destroy(self) -> None:
        if self._h:
            _lib.odma_paged_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def build(self, tables: Tables, host_len: Sequence[int], shuffle_seed: int, d_page_table: int,
              max_pages: int, stream: int = 0) -> None:
        _check(_lib.odma_paged_build(self._h, C.byref(tables), _i32arr(host_len), shuffle_seed,
                                     d_page_table, max_pages, stream or None), "odma_paged_build")

    def decode_attention(self, layer: int, q: int, q_heads: int, tables: Tables, d_page_table: int,
                         max_pages: int, out: int, lse: int = 0, stream: int = 0) -> None:
        _check(_lib.odma_decode_attention_paged(self._h, layer, q, q_heads, C.byref(tables),
                                                d_page_table, max_pages, out, lse or None,
                                                stream or None), "odma_decode_attention_paged")
