"""Invariants of the host-built split plan (no GPU)."""
import numpy as np
import pytest

from helpers import host_pool, lib
from paper_2512_09427_b200 import workloads as wl


def _plan(lens, kv_heads=4, ctas=148, max_len=32768 + 4096, headroom=0):
    buckets = [64, 256, 1024, 4096, 16384, max_len]
    tokens = sum(min(b for b in buckets if b >= L + headroom) for L in lens)
    w = wl.scaled(wl.config5(batch=1), pool_bytes=int(tokens * 1.3 + 64) * 2 * kv_heads * 128 * 2,
                  layers=1, kv_heads=kv_heads, max_len=max_len)
    pool = host_pool(w, plan_ctas=ctas, max_batch=max(1024, len(lens)))
    assert pool.set_buckets(buckets) == 0
    reqs = list(range(len(lens)))
    for r, L in zip(reqs, lens):
        rc, slab = pool.alloc(r, int(L) + headroom)
        assert rc == 0, rc
        if L > 1:
            assert pool.commit_step([r], [int(L) - 1]) == 0
    rc, t, words = pool.plan_host(reqs)
    assert rc == 0
    return pool, t, np.array(words, dtype=np.int64)


@pytest.mark.parametrize("lens", [
    [1], [64], [65], [17, 64, 100, 250], list(range(1, 200, 7)),
    list(wl.config2().context + 1), list(wl.config3().context + 1), list(wl.config5().context + 1),
    [16384] + [33] * 255,
])
@pytest.mark.parametrize("ctas", [1, 7, 148])
def test_plan_covers_every_tile_exactly_once_and_is_balanced(lens, ctas):
    hkv = 4
    pool, t, w = _plan(lens, hkv, ctas)
    n = len(lens)
    assert t.n == n and t.kv_tokens == sum(lens) and t.n_new_total == n and t.tile_tokens == 64
    assert t.one_new_each == 1
    assert list(w[t.off_len:t.off_len + n]) == list(lens)
    assert list(w[t.off_cu_new:t.off_cu_new + n + 1]) == list(range(n + 1))
    items = w[t.off_items:t.off_items + 8 * t.n_items].reshape(-1, 8)
    recs = w[t.off_cta:t.off_cta + 12 * t.n_ctas].reshape(-1, 12)
    # CTA c owns items [recs[c,0], recs[c,1]), shares are consecutive, and each record carries a
    # copy of its first item
    cta_begin = np.concatenate([recs[:, 0], recs[-1:, 1]])
    assert (recs[1:, 0] == recs[:-1, 1]).all() and (recs[:, 2:4] == 0).all()
    assert cta_begin[0] == 0 and cta_begin[-1] == t.n_items and (np.diff(cta_begin) >= 0).all()
    for c in range(t.n_ctas):
        if recs[c, 0] < recs[c, 1]:
            assert list(recs[c, 4:]) == list(items[recs[c, 0]])
    assert t.n_ctas <= ctas
    # within a CTA's share the pieces of split streams come first
    for c in range(t.n_ctas):
        d = items[cta_begin[c]:cta_begin[c + 1], 4] & 1
        assert list(d) == sorted(d)
    # slots number the pieces in (request, head, token) order; per stream they tile [0, len)
    # in order with no gap or overlap
    by_slot = items[np.argsort(items[:, 5])]
    assert list(by_slot[:, 5]) == list(range(t.n_items))
    cover = {}
    slabs = {r: pool.get_slab(r)[1] for r in range(n)}
    for req, head, tok0, ntok, flags, slot, row, ci in by_slot:
        direct = flags & 1
        assert ((flags >> 1) & 1) == (tok0 + ntok == lens[req])      # bit 1: the piece ends its stream
        assert ntok >= 1 and tok0 % 64 == 0
        base, cap = slabs[req][0], slabs[req][1]
        assert row == base * hkv + head * cap + tok0        # the documented row(head, t) formula
        assert (ci == -1) == bool(direct)
        cur = cover.get((req, head), 0)
        assert tok0 == cur
        cover[(req, head)] = tok0 + ntok
        whole = tok0 == 0 and ntok == lens[req]
        assert bool(direct) == whole
        if tok0 + ntok < lens[req]:
            assert ntok % 64 == 0                     # only a stream's last piece is ragged
    assert cover == {(r, h): lens[r] for r in range(n) for h in range(hkv)}
    # a stream's pieces have consecutive slots, in token order; streams come longest first
    seen, prev = [], None
    for req, head, tok0, *_ in by_slot:
        if (req, head) != prev:
            assert (req, head) not in seen
            seen.append((req, head))
            prev = (req, head)
    stream_lens = [lens[r] for r, _ in seen]
    assert [-(-L // 64) for L in stream_lens] == sorted((-(-L // 64) for L in stream_lens), reverse=True) or \
        stream_lens == sorted(stream_lens, reverse=True)
    comb = w[t.off_combine:t.off_combine + 4 * t.n_combine].reshape(-1, 4)
    split = {}
    for req, head, _, _, _, slot, _, _ in by_slot:
        split.setdefault((int(req), int(head)), []).append(int(slot))
    want = sorted((ks[0], r, h, len(ks)) for (r, h), ks in split.items() if len(ks) > 1)
    want = [(r, h, first, cnt) for first, r, h, cnt in want]
    assert [tuple(int(x) for x in c) for c in comb] == want
    for ci, (req, head, first, pieces) in enumerate(want):
        assert (by_slot[first:first + pieces, 7] == ci).all()
    # balance: shares are equal in cost: a tile costs 1, a stream start 1, a piece of a split (6 on top)
    # stream 2 on top; no share exceeds the average by more than a quarter (+ rounding)
    tiles = np.array([sum(-(-int(items[k, 3]) // 64) for k in range(cta_begin[c], cta_begin[c + 1]))
                      for c in range(t.n_ctas)])
    starts = np.array([sum(1 for k in range(cta_begin[c], cta_begin[c + 1]) if items[k, 2] == 0)
                       for c in range(t.n_ctas)])
    parts = np.array([sum(1 for k in range(cta_begin[c], cta_begin[c + 1]) if items[k, 4] & 1 == 0)
                      for c in range(t.n_ctas)])
    total = sum(-(-L // 64) for L in lens) * hkv
    assert tiles.sum() == total and starts.sum() == n * hkv
    cost = tiles + starts + 6 * parts
    if t.n_ctas > 1 and max(lens) > 128:
        assert cost.max() <= 1.25 * cost.sum() / ctas + 6, (cost.max(), cost.sum() / ctas)   # 6: a stream too short to split
    # pieces of split streams are never crumbs
    for req, head, tok0, ntok, flags, *_ in by_slot:
        if not (flags & 1) and lens[req] > 6 * 64:
            assert ntok >= 2 * 64 or tok0 + ntok == lens[req]
    assert t.words * 4 <= pool.tables_bytes(n)


def test_plan_rejects_bad_batches():
    odma = lib()
    pool, t, w = _plan([10, 20])
    assert pool.plan_host([0, 99])[0] == odma.ERR_UNKNOWN_REQ
    # request 0 sits at length 9 in a slab of... fill it to the brim, then one more does not fit
    rc, slab, ln = pool.get_slab(0)
    assert pool.commit_step([0], [slab[1] - ln]) == 0
    assert pool.plan_host([0, 1])[0] == odma.ERR_OVERFLOW
    assert pool.plan_host([0, 1], [0, 1])[0] == odma.OK


def test_a_decode_step_plan_is_reused_while_the_batch_only_grows_a_little():
    """Consecutive decode steps of the same batch keep the dealing of streams to CTAs; only the
    lengths (and with them the last piece of each stream) move.  After enough growth, or when a
    slab changes, the plan is made afresh."""
    lens = list(wl.config2().context + 1)
    hkv = 4
    pool, t0, w0 = _plan(lens, hkv, 148, headroom=64)   # _plan has committed len-1 tokens and planned +1
    reqs = list(range(len(lens)))

    def cover(t, w, cur):
        items = w[t.off_items:t.off_items + 8 * t.n_items].reshape(-1, 8)
        got = {}
        for req, head, tok0, ntok, flags, *_ in items[np.argsort(items[:, 5])]:
            assert got.get((req, head), 0) == tok0
            got[(req, head)] = tok0 + ntok
        assert got == {(r, h): cur[r] for r in reqs for h in range(hkv)}
        assert list(w[t.off_len:t.off_len + len(cur)]) == cur and t.kv_tokens == sum(cur)
        recs = w[t.off_cta:t.off_cta + 12 * t.n_ctas].reshape(-1, 12)
        for c in range(t.n_ctas):
            if recs[c, 0] < recs[c, 1]:
                assert list(recs[c, 4:]) == list(items[recs[c, 0]])
        return items

    base = cover(t0, w0, lens)
    cur = list(lens)
    for step in range(1, 40):
        assert pool.commit_step(reqs) == 0
        cur = [L + 1 for L in cur]
        rc, t, words = pool.plan_host(reqs)
        assert rc == 0
        items = cover(t, np.array(words, dtype=np.int64), cur)
        same = items.shape == base.shape and np.array_equal(items[:, [0, 1, 2, 4, 5, 6, 7]], base[:, [0, 1, 2, 4, 5, 6, 7]])
        if step <= 32:
            assert same, step                      # same pieces on the same CTAs, longer ends
        else:
            base = items if not same else base     # a fresh plan may cut elsewhere
    # a request that moved to another slab invalidates the cached plan at once
    rc, slab, ln = pool.get_slab(0)
    rc, slab2, mig = pool.ensure_capacity(0, slab[1] + 1)        # beyond its slab: moves to the Large Bucket
    assert rc == 0 and mig == 1
    rc, t, words = pool.plan_host(reqs)
    assert rc == 0
    items = cover(t, np.array(words, dtype=np.int64), cur)
    row0 = items[(items[:, 0] == 0) & (items[:, 1] == 0) & (items[:, 2] == 0)][0, 6]
    assert row0 == slab2[0] * hkv


def test_plan_never_outgrows_the_table_it_was_sized_for():
    """Random length mixes and CTA counts: the words a plan writes stay within
    odma_tables_bytes (items <= streams + ctas, cut streams <= min(streams, ctas))."""
    rng = np.random.default_rng(5)
    odma = lib()
    for trial in range(300):
        n = int(rng.integers(1, 40))
        ctas = int(rng.integers(1, 200))
        kind = trial % 3
        if kind == 0:
            lens = rng.integers(1, 200, size=n)
        elif kind == 1:
            lens = np.clip(np.rint(np.exp(rng.normal(6, 1.2, size=n))), 1, 16000).astype(int)
        else:
            lens = rng.choice([1, 63, 64, 65, 4096, 16000], size=n)
        w = wl.scaled(wl.config1("a"), pool_bytes=1 << 30, max_len=16384, context=np.asarray(lens, dtype=np.int64),
                      predicted=np.asarray(lens, dtype=np.int64) + 1)
        pool = host_pool(w, plan_ctas=ctas, max_batch=64)
        assert pool.set_buckets([16384]) == 0
        reqs = list(range(n))
        for r in reqs:
            assert pool.alloc(r, int(lens[r]) + 1)[0] == 0
            assert pool.commit_step([r], [int(lens[r])]) == 0
        rc, t, words = pool.plan_host(reqs)
        assert rc == 0
        assert t.words * 4 <= pool.tables_bytes(n)
        assert t.n_items <= n * w.kv_heads + ctas and t.n_combine <= min(n * w.kv_heads, ctas)
