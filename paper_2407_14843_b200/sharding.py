"""Splitting a batch of independent instances over ranks (one GPU each).

Instances never interact, so the solve path needs no collective: every rank
solves a contiguous block of the batch against replicated latency tables.  A
single ``all_gather`` of the small result arrays assembles the full answer
when one buffer is wanted.
"""
from __future__ import annotations

from typing import Callable, Dict, Tuple

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


def solve_sharded(wl, solve_fn: Callable, group=None) -> Dict[str, torch.Tensor]:
    """Solves one batch across the ranks of a process group: every rank takes its
    ``shard_range`` block of ``wl`` (a ``workloads.Workload``; the latency tables are
    replicated, no instance data crosses ranks), solves it with ``solve_fn(block)`` and
    the result arrays are all-gathered, so every rank returns the full-batch arrays in
    instance order.

    ``solve_fn`` takes a Workload and returns a mapping with the keys of ``RESULT_KEYS``
    (torch tensors or numpy arrays, rows = the block's instances): on a GPU rank
    ``lambda block: solver.solve(block)[0]`` with the rank's device current.  The only
    collective is the gather of the results (``N * (3 * S + 3) * 4`` bytes)."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    start, stop = shard_range(wl.n_instances, rank, world)
    local = solve_fn(wl.take(stop - start, start))
    local = {k: torch.as_tensor(local[k]) for k in RESULT_KEYS}
    return gather_results(local, wl.n_instances, group)
