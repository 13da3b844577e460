"""Bucket configuration kept consistent across the replicas of a node (Section III-E: a cluster
manager synchronises the logical bucket configuration of the devices).

Each replica owns its pool and allocator (the attention path shards by request, nothing of it is
exchanged).  What the replicas share is the evidence the boundaries are derived from: with
`cluster_observe = 1` a pool keeps the realised lengths of its completions in an outbox instead of
its window; `sync()` gathers every replica's outbox and feeds the concatenation, in rank order, to
every pool (`odma_observe`), so all windows hold the same sequence and Eq. 2 gives the same
boundaries everywhere.  The exchange is a few integers per completed request over the process
group the caller passes in (gloo or NCCL); it is host-side and off the decode path.
"""
from __future__ import annotations

from typing import List, Optional


class ClusterManager:
    def __init__(self, pool, group=None):
        """`pool`: this replica's odma.Pool, created with cluster_observe = 1.  `group`: a
        torch.distributed process group (None = the default group; a single process works too)."""
        self.pool = pool
        self.group = group
        self.rounds = 0

    def sync(self) -> List[int]:
        """One exchange round: returns the merged lengths that were observed (identical on every rank)."""
        import torch.distributed as dist
        mine = self.pool.drain_observations()
        if dist.is_available() and dist.is_initialized():
            world = dist.get_world_size(self.group)
            parts: List[Optional[List[int]]] = [None] * world
            dist.all_gather_object(parts, mine, group=self.group)
        else:
            parts = [mine]
        merged = [x for part in parts for x in part]
        if merged:
            self.pool.observe(merged)
        self.pool.recal_flush()
        self.rounds += 1
        return merged

    def boundaries(self):
        return self.pool.get_buckets()
