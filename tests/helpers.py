"""Shared test helpers: adapters that give the library's allocator and the CPU checker's
allocator the same face, and a lock-step wrapper that compares them at every event."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle as ora
from paper_2512_09427_b200 import workloads as wl


def lib():
    from paper_2512_09427_b200 import odma
    return odma


# configuration fields applied to every pool a test creates (a module's fixture may set, say,
# the decode kernel to run the same tests on both tensor-core kernels)
CFG_DEFAULTS = {}


def make_cfg(w: wl.Workload, **over):
    odma = lib()
    cfg = odma.config_default()
    over = {**CFG_DEFAULTS, **over}
    cfg.safety_pct, cfg.max_len, cfg.granule = w.safety_pct, w.max_len, w.granule
    cfg.window, cfg.refresh = w.window, w.refresh
    pn, pd = w.quantiles
    cfg.n_levels = len(pn)
    for i, x in enumerate(pn):
        cfg.p_num[i] = x
    cfg.p_den = pd
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


def oracle_allocator(w: wl.Workload, **over) -> ora.Allocator:
    pn, pd = w.quantiles
    args = dict(safety_pct=w.safety_pct, max_len=w.max_len, granule=w.granule, window=w.window,
                refresh=w.refresh, p_num=pn, p_den=pd)
    args.update(over)
    return ora.Allocator(w.pool_bytes, w.layers, w.kv_heads, w.head_dim, w.elem_bytes, **args)


def pool_dtype(w: wl.Workload) -> int:
    odma = lib()
    if w.kv_dtype == "e4m3":
        return odma.DTYPE_FP8_E4M3
    return odma.DTYPE_BF16 if w.dtype == torch.bfloat16 else odma.DTYPE_F32


def host_pool(w: wl.Workload, **over):
    """A bookkeeping-only pool (no device memory)."""
    odma = lib()
    dt = pool_dtype(w)
    return odma.Pool(0, w.pool_bytes, w.layers, w.kv_heads, w.head_dim, dt, make_cfg(w, **over))


class LockStep:
    """Feeds every allocator call to the library and to the checker and asserts equal answers."""

    def __init__(self, pool, oracle: ora.Allocator, stream: int = 0):
        self.pool, self.oracle, self.stream = pool, oracle, stream
        self.events = 0

    def alloc(self, req, predicted):
        rc_o, slab_o = self.oracle.reserve(req, predicted)
        rc_p, slab_p = self.pool.alloc(req, predicted)
        assert rc_p == rc_o, ("alloc", req, predicted, rc_p, rc_o)
        assert slab_p == slab_o, ("alloc", req, predicted, slab_p, slab_o)
        self.events += 1
        return slab_p[:4] if rc_p == 0 else None

    def alloc_uncertain(self, req, l_hat, u):
        rc_o, slab_o = self.oracle.reserve_uncertain(req, l_hat, u)
        rc_p, slab_p = self.pool.alloc_uncertain(req, l_hat, u)
        assert (rc_p, slab_p) == (rc_o, slab_o), ("alloc_uncertain", req, l_hat, u, rc_p, slab_p, rc_o, slab_o)
        self.events += 1
        return rc_p, slab_p

    def ensure_rc(self, req, need):
        rc_o, slab_o, mig_o = self.oracle.ensure_capacity(req, need)
        rc_p, slab_p, mig_p = self.pool.ensure_capacity(req, need, self.stream)
        assert (rc_p, slab_p, mig_p) == (rc_o, slab_o, mig_o), ("ensure", req, need, rc_p, slab_p, mig_p,
                                                              rc_o, slab_o, mig_o)
        self.events += 1
        return rc_p, slab_p, mig_p

    def ensure(self, req, need):
        rc, slab, mig = self.ensure_rc(req, need)
        if rc == 2:                      # ODMA_ERR_NOMEM: the caller preempts the request
            return None
        assert rc == 0, ("ensure", req, need, rc)
        return slab[:4], mig

    def commit(self, reqs, n_new):
        reqs = list(reqs)
        for r in reqs:
            assert self.oracle.add_len(r, n_new) == 0
        assert self.pool.commit_step(reqs, [n_new] * len(reqs)) == 0

    def free(self, req):
        rc_o = self.oracle.release(req)
        rc_p = self.pool.free(req)
        assert rc_p == rc_o == 0, ("free", req, rc_p, rc_o)
        assert self.pool.get_buckets() == self.oracle.get_buckets()
        self.events += 1

    def buckets(self):
        b = self.pool.get_buckets()
        assert b == self.oracle.get_buckets()
        return b

    def check_stats(self):
        sp, so = self.pool.get_stats(), self.oracle.stats()
        for k_o, k_p in [("live", "live"), ("reserved_live", "reserved_live"), ("used_live", "used_live"),
                         ("completed", "completed"), ("sum_len_completed", "sum_len_completed"),
                         ("sum_cap_completed", "sum_cap_completed"), ("migrations", "migrations"),
                         ("nomem", "nomem"), ("routed_large", "routed_large"),
                         ("safety_live", "safety_live"), ("safety_peak", "safety_peak"),
                         ("observed", "observed")]:
            assert sp[k_p] == so[k_o], (k_p, sp[k_p], so[k_o])
        assert (sp["total_tokens"], sp["safety_tokens"], sp["main_tokens"]) == \
               (self.oracle.T, self.oracle.S, self.oracle.M)
        return sp


def warm_up(ls: LockStep, lengths: np.ndarray, first_req: int = 1 << 40):
    """Log realised lengths (alloc, grow to the length, free) so the boundaries are learned."""
    for i, L in enumerate(lengths):
        r = first_req + i
        slab = ls.alloc(r, int(L))
        assert slab is not None
        ls.commit([r], int(L))
        ls.free(r)


# ---------------------------------------------------------------------------------------------
# GPU session: one device pool driven through the C ABI, mirrored by the CPU checker
# ---------------------------------------------------------------------------------------------

class Session:
    """A device pool plus its CPU mirror (checker allocator + checker KV store).

    Every allocator call goes to both sides in lock step; every row appended on the device is
    also handed to the checker's own store, so attention can be compared without reading the
    pool back.  Inputs come from the seeded generators in `workloads`.
    """

    def __init__(self, w: wl.Workload, fill=None, mirror_kv=True, **cfg_over):
        odma = lib()
        self.odma, self.w = odma, w
        self.dev = torch.device("cuda:0")
        self.gen_dev = self.dev          # where the seeded inputs are generated ("cpu": no generator kernels on the GPU)
        self.dt = pool_dtype(w)
        self.e4m3 = w.kv_dtype == "e4m3"
        self.mem = torch.empty(w.pool_bytes, dtype=torch.uint8, device=self.dev)
        if fill is not None:
            self.mem.view(torch.int16).fill_(fill)
        else:
            self.mem.zero_()
        self.stream = torch.cuda.current_stream().cuda_stream
        self.cfg = make_cfg(w, **cfg_over)
        self.pool = odma.Pool(self.mem.data_ptr(), w.pool_bytes, w.layers, w.kv_heads, w.head_dim,
                              self.dt, self.cfg)
        self.ls = LockStep(self.pool, oracle_allocator(w), self.stream)
        self.k_scale, self.v_scale = wl.e4m3_scales(w.layers) if self.e4m3 else (None, None)
        if self.e4m3:
            self.pool.set_kv_scales(self.k_scale, self.v_scale)
        self.kv = ora.KVStore(w.layers, w.kv_heads, w.head_dim, ora.dtype_code(w.dtype), kv_e4m3=self.e4m3,
                              k_scale=self.k_scale, v_scale=self.v_scale) if mirror_kv else None
        self.table = torch.empty(self.pool.tables_bytes(self.cfg.max_batch), dtype=torch.uint8, device=self.dev)
        self.lens = {}
        st = self.pool.get_stats()
        self.T = st["total_tokens"]

    # -- allocation ---------------------------------------------------------------------------
    def admit(self, reqs, predicted):
        for r, p in zip(reqs, predicted):
            assert self.ls.alloc(int(r), int(p)) is not None
            self.lens[int(r)] = 0

    def tables(self, reqs, n_new=None):
        return self.pool.build_tables([int(r) for r in reqs], self.table.data_ptr(), self.table.numel(),
                                      self.stream, n_new)

    # -- data ---------------------------------------------------------------------------------
    def rows(self, layer, req, kind, t0, t1, scale=1.0):
        x = wl.kv_rows(self.w.seed, layer, req, kind, t0, t1, self.w.kv_heads, self.w.head_dim,
                       self.w.dtype, self.gen_dev)
        x = x if scale == 1.0 else (x.float() * scale).to(self.w.dtype)
        return x.to(self.dev)

    def append(self, reqs, n_new, layers=None, scale=1.0):
        """Append n_new[i] generated tokens to every request, on all layers; commit lengths."""
        reqs = [int(r) for r in reqs]
        n_new = [int(x) for x in n_new]
        for r, k in zip(reqs, n_new):
            self.ls.ensure(r, self.lens[r] + k)
        t = self.tables(reqs, n_new)
        for layer in (range(self.w.layers) if layers is None else layers):
            ks = [self.rows(layer, r, wl.KIND_K, self.lens[r], self.lens[r] + k, scale) for r, k in zip(reqs, n_new)]
            vs = [self.rows(layer, r, wl.KIND_V, self.lens[r], self.lens[r] + k) for r, k in zip(reqs, n_new)]
            k_new, v_new = torch.cat(ks).contiguous(), torch.cat(vs).contiguous()
            self.pool.append_kv(layer, t, k_new.data_ptr(), v_new.data_ptr(), self.stream)
            if self.kv is not None:
                for r, kk, vv in zip(reqs, ks, vs):
                    if kk.shape[0]:
                        self.kv.append(r, layer, kk, vv)
        torch.cuda.synchronize()
        for r, k in zip(reqs, n_new):
            self.ls.commit([r], k)
            self.lens[r] += k
        return t

    def queries(self, layer, reqs, q_heads, step=0, scale=1.0):
        q = torch.stack([wl.q_rows(self.w.seed, layer, int(r), step, q_heads, self.w.head_dim,
                                   self.w.dtype, self.gen_dev) for r in reqs]).contiguous()
        q = q if scale == 1.0 else (q.float() * scale).to(self.w.dtype)
        return q.to(self.dev)

    def decode_step(self, reqs, q_heads, layers=None, step=0, want_lse=True, scale=1.0):
        """One decode step: ensure room, build tables, then per layer append one token and attend.
        Returns {layer: (out, lse, q)} as device tensors; lengths are committed."""
        reqs = [int(r) for r in reqs]
        for r in reqs:
            self.ls.ensure(r, self.lens[r] + 1)
        t = self.tables(reqs)
        res = {}
        for layer in (range(self.w.layers) if layers is None else layers):
            ks = [self.rows(layer, r, wl.KIND_K, self.lens[r], self.lens[r] + 1, scale) for r in reqs]
            vs = [self.rows(layer, r, wl.KIND_V, self.lens[r], self.lens[r] + 1) for r in reqs]
            k_new, v_new = torch.cat(ks).contiguous(), torch.cat(vs).contiguous()
            q = self.queries(layer, reqs, q_heads, step, scale)
            out = torch.full_like(q, float("nan"))
            lse = torch.full((len(reqs), q_heads), float("nan"), dtype=torch.float32, device=self.dev)
            self.pool.append_kv(layer, t, k_new.data_ptr(), v_new.data_ptr(), self.stream)
            self.pool.decode_attention(layer, q.data_ptr(), q_heads, t, out.data_ptr(),
                                       lse.data_ptr() if want_lse else 0, self.stream)
            if self.kv is not None:
                for r, kk, vv in zip(reqs, ks, vs):
                    self.kv.append(r, layer, kk, vv)
            res[layer] = (out, lse, q)
        torch.cuda.synchronize()
        assert self.pool.check_status(self.stream) == 0
        self.ls.commit(reqs, 1)
        for r in reqs:
            self.lens[r] += 1
        self.last_tables = t
        return res

    # -- checks -------------------------------------------------------------------------------
    def oracle_out(self, layer, reqs, q, q_heads):
        return self.kv.decode_attention(layer, [int(r) for r in reqs], q, q_heads, want_lse=True)

    def pool_rows(self, layer, kv, req, head=None):
        """The request's rows read back from the device pool through the documented formula:
        [len, kv_heads, head_dim] in token-major order (8-bit pools: the codes, uint8)."""
        rc, slab, ln = self.pool.get_slab(int(req))
        assert rc == 0
        base, cap = slab[0], slab[1]
        w = self.w
        n_elems = w.layers * 2 * self.T * w.kv_heads * w.head_dim
        arr = self.mem.view(torch.uint8 if self.e4m3 else w.dtype)[:n_elems].view(w.layers * 2, self.T * w.kv_heads, w.head_dim)[layer * 2 + kv]
        heads = [arr[base * w.kv_heads + h * cap: base * w.kv_heads + h * cap + ln] for h in range(w.kv_heads)]
        return torch.stack(heads, dim=1)


def attention_errors(out, ref):
    """(max abs error, relative L2 error) of a device result against the fp64 reference."""
    o = out.detach().double().cpu().numpy()
    err = np.abs(o - ref).max()
    rel = np.linalg.norm((o - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300)
    return float(err), float(rel)


# tolerances of the benchmark spec: bf16 inputs / fp32 accumulation, and fp32 inputs
BF16_MAX_ABS, BF16_REL_L2 = 1e-2, 5e-3
F32_MAX_ABS = 1e-5


def assert_close(out, ref, dtype, what=""):
    err, rel = attention_errors(out, ref)
    if dtype == torch.bfloat16:
        assert err <= BF16_MAX_ABS and rel <= BF16_REL_L2, (what, err, rel)
    else:
        assert err <= F32_MAX_ABS, (what, err, rel)
    return err, rel
