"""Admission / serving simulator, checker side (plain Python, one token at a time).

TEST INFRASTRUCTURE ONLY: the slow, plain statement of what the library's native simulator
(odma_sim_run) must compute; only the tests call it, and it shares no code with the library.

What is simulated (Section V of the paper: requests arrive by a Poisson process and share one
KV-cache pool; reported are KV-cache utilisation = sum of actual KV use over sum of reserved
KV, and throughput in output tokens per second): a single model replica decoding in lock
step.  Three reservation policies run on the same request trace:

  STATIC   every admitted request reserves max_len tokens (the worst-case pre-allocation of
           the static baseline, Sections I and V)
  PAGED    16-token pages taken on demand (the PagedAttention accounting the paper contrasts
           itself with, Sections I, II-A)
  ODMA     the bucket allocator of Section III through the checker's brute-force Allocator:
           slab = predicted-length bucket (with the uncertainty inflation and routing of
           Section III-B when the request carries an uncertainty), overflow = allocate-and-
           copy migration into the Large Bucket (Sections III-D, IV-C)

Rules (where the paper is silent, the reading is stated):
  * time is an integer number of nanoseconds; the prompt is in the slab at admission
    (prefill is not timed); a decode step lasts
        layers * (base_ns + kv_tokens * ps_per_token // 1000)
    with kv_tokens = the keys attended this step over all generating requests (the attention
    path's cost model: a fixed part per launch plus streaming time per KV token);
  * admission is first come first served and stops at the first request that does not fit (no
    overtaking), at max_batch live requests, or at a request that has not arrived yet; with
    nobody live the clock jumps to the next arrival;
  * a live request that cannot get room for its next token (no free page / no Large Bucket
    slab) stalls for the step; when every live request is stalled, the youngest is preempted
    (its memory freed, its progress lost, it rejoins the head of the queue) and nothing is
    admitted until a live request has completed (else the preempted request would come
    straight back and the pool would thrash);
  * a request whose prompt cannot be placed even in an empty pool, or that stalls while it is
    the only live request, can never finish and is dropped (failed).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence

STATIC, PAGED, ODMA = 0, 1, 2
PAGE = 16


@dataclass
class SimRequest:
    arrival_ns: int
    prompt: int          # KV tokens present at admission
    total: int           # KV tokens when the request completes (prompt + generated)
    predicted: int       # predicted total (what the allocator is told)
    u_permille: int = -1  # predictor uncertainty in thousandths, -1: none (plain reserve)


@dataclass
class SimResult:
    completed: int = 0
    failed: int = 0
    tokens_out: int = 0       # tokens generated, those of later preempted runs included ...
    tokens_lost: int = 0      # ... which are counted here as well
    steps: int = 0
    makespan_ns: int = 0
    sum_actual: int = 0       # over completed requests: KV tokens used ...
    sum_reserved: int = 0     # ... and reserved when they completed (utilisation = ratio)
    conc_time: int = 0        # integral of live requests over time (ns)
    reserved_time: int = 0    # integral of reserved tokens over time
    used_time: int = 0        # integral of used tokens over time
    migrations: int = 0
    preemptions: int = 0
    stalls: int = 0
    deferred: int = 0         # admission attempts that found no room
    log: List[tuple] = field(default_factory=list)


def _ceil_page(x: int) -> int:
    return -(-x // PAGE) * PAGE


def simulate(policy: int, total_tokens: int, max_len: int, requests: Sequence[SimRequest], max_batch: int,
             layers: int, base_ns: int, ps_per_token: int, allocator=None) -> SimResult:
    """`allocator`: a fresh oracle.Allocator for ODMA (its pool geometry is the pool);
    `total_tokens`: the pool size the other two policies account against."""
    res = SimResult()
    queue = list(range(len(requests)))          # request indices, head first
    live: List[int] = []                        # in admission order
    length = {}                                 # live request -> KV tokens held
    reserved = {}                               # live request -> tokens reserved
    free = total_tokens                         # STATIC / PAGED only
    now = 0
    hold = False                                # no admission between a preemption and the next completion

    def release(r):
        nonlocal free
        if policy == ODMA:
            assert allocator.release(r) == 0
        else:
            free += reserved[r]
        del length[r], reserved[r]

    while queue or live:
        # ---- admission
        while queue and len(live) < max_batch and not (hold and live):
            r = queue[0]
            q = requests[r]
            if q.arrival_ns > now:
                if live:
                    break
                now = q.arrival_ns               # idle: jump to the next arrival
            ok = True
            if policy == STATIC:
                need = max_len
                if need > total_tokens or q.total > max_len:
                    res.failed += 1
                    queue.pop(0)
                    continue
                if free < need:
                    ok = False
                else:
                    free -= need
                    reserved[r] = need
            elif policy == PAGED:
                need = _ceil_page(q.prompt)
                if _ceil_page(q.total) > total_tokens:
                    res.failed += 1
                    queue.pop(0)
                    continue
                if free < need:
                    ok = False
                else:
                    free -= need
                    reserved[r] = need
            else:
                if q.u_permille >= 0:
                    rc, slab = allocator.reserve_uncertain(r, q.predicted, q.u_permille)
                else:
                    rc, slab = allocator.reserve(r, q.predicted)
                if rc == 2:                      # no memory
                    ok = False
                else:
                    assert rc == 0, rc
                    cap = slab[1]
                    if q.prompt > cap:           # predicted below the prompt: grow at once
                        rc, slab, mig = allocator.ensure_capacity(r, q.prompt)
                        if rc != 0:
                            assert allocator.release(r) == 0
                            if not live:
                                res.failed += 1
                                queue.pop(0)
                                continue
                            ok = False
                        else:
                            res.migrations += mig
                            cap = slab[1]
                    if ok:
                        assert allocator.add_len(r, q.prompt) == 0
                        reserved[r] = cap
            if not ok:
                res.deferred += 1
                if not live:                     # nothing will ever free memory for it
                    res.failed += 1
                    queue.pop(0)
                    continue
                break
            queue.pop(0)
            live.append(r)
            length[r] = q.prompt
            res.log.append(("admit", now, r, reserved[r]))
        if not live:
            continue
        # ---- one decode step: room for each live request's next token
        gen = []
        for r in live:
            L = length[r]
            if policy == PAGED:
                if L + 1 > reserved[r]:
                    if free < PAGE:
                        res.stalls += 1
                        continue
                    free -= PAGE
                    reserved[r] += PAGE
            elif policy == ODMA:
                if L + 1 > reserved[r]:
                    rc, slab, mig = allocator.ensure_capacity(r, L + 1)
                    if rc != 0:
                        assert rc == 2, rc
                        res.stalls += 1
                        continue
                    res.migrations += mig
                    reserved[r] = slab[1]
            gen.append(r)
        if not gen:
            r = live.pop()                       # everybody stalled: the youngest goes back
            res.tokens_lost += length[r] - requests[r].prompt
            alone = not live
            release(r)
            if alone:                            # it had the pool to itself and still could not grow
                res.failed += 1
                res.log.append(("fail", now, r, 0))
                hold = False
                continue
            hold = True
            queue.insert(0, r)
            res.preemptions += 1
            res.log.append(("preempt", now, r, 0))
            continue
        kv_tokens = sum(length[r] + 1 for r in gen)
        step_ns = layers * (base_ns + kv_tokens * ps_per_token // 1000)
        now += step_ns
        for r in gen:
            length[r] += 1
            if policy == ODMA:
                assert allocator.add_len(r, 1) == 0
        res.steps += 1
        res.tokens_out += len(gen)
        res.conc_time += len(live) * step_ns
        res.reserved_time += sum(reserved[r] for r in live) * step_ns
        res.used_time += sum(length[r] for r in live) * step_ns
        # ---- completions
        for r in [r for r in live if length[r] >= requests[r].total]:
            res.completed += 1
            res.sum_actual += length[r]
            res.sum_reserved += reserved[r]
            res.log.append(("done", now, r, reserved[r]))
            live.remove(r)
            release(r)
            hold = False
    res.makespan_ns = now
    return res
