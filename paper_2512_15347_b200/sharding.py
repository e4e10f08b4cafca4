"""Multi-GPU layout of a rollout batch: prompt groups are independent (selection and advantages
are per group, noise is keyed by the global trajectory id), so a job is split by groups and no
data-path collective is needed.  Only timing and optional result gathering use the process group.
"""
from __future__ import annotations

from typing import Tuple


def group_shard(n_groups_total: int, world: int, rank: int) -> Tuple[int, int]:
    """(first group, number of groups) of `rank` when n_groups_total groups are dealt out in
    contiguous blocks; the first n_groups_total % world ranks hold one group more."""
    if world < 1 or not 0 <= rank < world or n_groups_total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_groups_total, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def weak_shard(groups_per_rank: int, rank: int) -> Tuple[int, int]:
    """Weak scaling: every rank runs groups_per_rank groups; returns (group_offset, count)."""
    return rank * groups_per_rank, groups_per_rank


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Largest value over all ranks of the default process group (identity without one)."""
    if dist is None or not dist.is_initialized():
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def all_gather_groups(t, dist=None):
    """Concatenates a per-group (or per-trajectory) tensor over ranks in rank order, i.e. in global
    group order for contiguous shards of equal size.  The only collective the sharded rollout can
    need: a few KB of advantages / statistics when one rank wants the whole batch."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return t
    import torch
    parts = [torch.empty_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, t.contiguous())
    return torch.cat(parts, dim=0)
