"""Head-sharded multi-GPU use of the routed-attention layer.

Heads are independent units (the select of a head needs only that head's features, the
masks are geometry), so a layer splits over ranks by heads with no exchange inside the op.
`shard_heads` asks the library for the partition (longest-processing-time-first packing of
the heads by the attention work of their routes, `vorta_shard_heads`); `HeadShardedLayer`
runs one rank's share through a plan over its own heads; `all_gather_heads` puts the full
output together on every rank with one plain all-gather into local memory, for callers whose
next operator is not head-sharded.  One process per GPU, `torch.distributed` for the plumbing.
"""
from __future__ import annotations

from dataclasses import replace
from typing import List, Sequence, Tuple

import numpy as np
import torch

from . import binding as vb


def shard_heads(wl, n_ranks: int) -> Tuple[np.ndarray, np.ndarray]:
    """(rank_of_head int32 [heads], rank_flops float64 [n_ranks]) for the workload's routes.

    Host-only: needs no GPU."""
    plan = vb.Plan.from_workload(wl, host_only=True)
    try:
        return vb.vorta_shard_heads(plan.handle, wl.heads, n_ranks)
    finally:
        plan.close()


def heads_of_rank(rank_of_head: Sequence[int], rank: int) -> List[int]:
    return [h for h, r in enumerate(rank_of_head) if int(r) == rank]


def local_workload(wl, heads: Sequence[int]):
    """The workload restricted to `heads` (ascending), as one rank sees it."""
    heads = list(heads)
    return replace(wl, name=f"{wl.name}[{len(heads)} heads]", heads=len(heads),
                   routes=tuple(wl.routes[h] for h in heads))


class HeadShardedLayer:
    """One rank's share of a layer.

    `heads` are the global indices of the heads this rank owns; Q, K, V, O passed to
    `__call__` are the rank's slices `[B, len(heads), L, d]` (head-sharded inputs, as after an
    all-to-all upstream)."""

    def __init__(self, wl, rank: int, world_size: int, device: int = -1):
        self.wl, self.rank, self.world_size = wl, rank, world_size
        self.rank_of_head, self.rank_flops = shard_heads(wl, world_size)
        self.heads = heads_of_rank(self.rank_of_head, rank)
        self.local = local_workload(wl, self.heads)
        self._device = device
        self.plan = None  # created at the first call: the partition itself needs no GPU

    def close(self):
        if self.plan is not None:
            self.plan.close()
            self.plan = None

    def __call__(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, O: torch.Tensor) -> torch.Tensor:
        if not self.heads:
            return O
        if self.plan is None:
            self.plan = vb.Plan.from_workload(self.local, device=self._device)
        self.plan.routed_attention(Q, K, V, O)
        return O

    def take_local(self, full: torch.Tensor) -> torch.Tensor:
        """This rank's heads of a `[B, heads, L, d]` tensor (a copy, contiguous)."""
        return full[:, self.heads].contiguous()


def all_gather_heads(local_O: torch.Tensor, rank_of_head: Sequence[int], group=None) -> torch.Tensor:
    """Assemble `[B, heads, L, d]` on every rank from the ranks' `[B, heads_r, L, d]` outputs.

    One all-gather of equal-sized buffers (ranks with fewer heads pad), then a local
    reordering by `rank_of_head`; nothing reads another GPU's memory directly."""
    import torch.distributed as dist

    world = dist.get_world_size(group)
    counts = [sum(1 for r in rank_of_head if int(r) == k) for k in range(world)]
    most = max(counts)
    B, _, L, d = local_O.shape
    padded = local_O.new_zeros((B, most, L, d))
    padded[:, : local_O.shape[1]] = local_O
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    out = local_O.new_empty((B, len(rank_of_head), L, d))
    for k in range(world):
        heads = heads_of_rank(rank_of_head, k)
        if heads:
            out[:, heads] = parts[k][:, : len(heads)]
    return out
