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


def all_ranks_ok(ok: bool, dist=None, device=None) -> bool:
    """True only if every rank passes True: lets all ranks take the same branch after a step that
    may fail on some of them (e.g. pinning tens of GB of host memory), so that none is left alone
    in a later collective."""
    return max_over_ranks(0.0 if ok else 1.0, dist, device) == 0.0


def all_gather_groups(t, dist=None, group=None):
    """Concatenates a per-group (or per-trajectory) tensor over ranks in rank order, i.e. in global
    group order for contiguous shards.  Shards may differ in their first dimension (group_shard
    hands the first ranks one group more; a rank may even hold nothing): the lengths are exchanged
    first, every rank pads to the longest, and the padding is cut away after the gather.  The only
    collective the sharded rollout can need: a few KB of advantages / statistics when one rank
    wants the whole batch."""
    if dist is None or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return t
    import torch
    world = dist.get_world_size(group)
    t = t.contiguous()
    n_local = torch.tensor([t.shape[0]], dtype=torch.int64, device=t.device)
    lengths = [torch.empty_like(n_local) for _ in range(world)]
    dist.all_gather(lengths, n_local, group=group)
    lengths = [int(v.item()) for v in lengths]
    longest = max(lengths)
    if longest == 0:
        return t
    padded = t
    if t.shape[0] < longest:
        padded = torch.zeros((longest,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        padded[: t.shape[0]] = t
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    return torch.cat([p[:n] for p, n in zip(parts, lengths)], dim=0)
