"""Splitting a batch of independent instances over ranks (one GPU each).

Instances never interact, so the solve path needs no collective: every rank
solves a contiguous block of the batch against replicated latency tables.  A
single ``all_gather`` of the small result arrays assembles the full answer
when one buffer is wanted.
"""
from __future__ import annotations

from typing import Dict, Tuple

import torch
import torch.distributed as dist

RESULT_KEYS = ("h", "c", "b", "total_cost", "latency_buckets", "status")


def shard_range(n_instances: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block [start, stop) of rank ``rank``; sizes differ by at most one."""
    if not (0 <= rank < world) or n_instances < 0:
        raise ValueError("bad rank/world/n_instances")
    base, extra = divmod(n_instances, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def gather_results(local: Dict[str, torch.Tensor], n_instances: int, group=None) -> Dict[str, torch.Tensor]:
    """All-gathers per-rank result arrays (rows = this rank's instances, in
    ``shard_range`` order) into full-batch arrays on every rank."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    longest = shard_range(n_instances, 0, world)
    longest = longest[1] - longest[0]
    out = {}
    for k in RESULT_KEYS:
        t = local[k]
        pad_shape = (longest,) + tuple(t.shape[1:])
        padded = torch.zeros(pad_shape, dtype=t.dtype, device=t.device)
        padded[: t.shape[0]] = t
        parts = [torch.empty_like(padded) for _ in range(world)]
        dist.all_gather(parts, padded, group=group)
        rows = []
        for r in range(world):
            a, b = shard_range(n_instances, r, world)
            rows.append(parts[r][: b - a])
        out[k] = torch.cat(rows, dim=0)
    del rank
    return out
