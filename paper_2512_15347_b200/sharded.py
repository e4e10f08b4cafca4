"""Group-sharded multi-GPU driver: one process per GPU, every process runs the Expand-and-Prune
rollout of its own contiguous block of prompt groups.

Prompt groups are independent - the selection (Eq. ovf) and the advantages (Eq. advK) are per
group and the noise of a trajectory is keyed by its global id - so the rollout itself needs no
exchange between GPUs: a rank's handle is created with the index of its first group
(``group_offset``) and produces exactly the rows the unsharded rollout would.  The process group
is used for two things only: the maximum over ranks of a device time, and ``gather()``, an
all-gather of the few KB of per-group results (advantages, group mean / std, rewards, trajectory
ids) for a trainer that wants the whole batch on every rank.

Launch with ``python -m torch.distributed.run --nproc-per-node N -m paper_2512_15347_b200.sharded
--workload sd3`` (rendezvous on 127.0.0.1); without a launcher the module runs as a single rank.
"""
from __future__ import annotations

import argparse
import json
import os
from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple

import torch

from . import sharding


@dataclass
class GatheredResults:
    """Per-group results of the whole job, in global group order, on every rank."""
    adv: torch.Tensor        # [G_total * K] fp32
    rewards: torch.Tensor    # [G_total * K] fp32
    mean: torch.Tensor       # [G_total] fp32
    std: torch.Tensor        # [G_total] fp32
    traj_id: torch.Tensor    # [G_total * K] int32, global trajectory ids of the survivors
    shards: List[Tuple[int, int]]   # (first group, groups) of every rank


def _default_factory(*args, **kw):
    from .rollout import Rollout
    return Rollout(*args, **kw)


class ShardedRollout:
    """The rollout of ``total_groups`` prompt groups dealt out over the ranks of a process group.

    Rank r owns the groups ``sharding.group_shard(total_groups, world, r)`` (contiguous blocks,
    the first ``total_groups % world`` ranks one group more; a rank may own none).  ``local`` is
    that rank's ``Rollout`` (None without groups), built with the shard's ``group_offset`` so that
    trajectory ids - and with them the noise - are those of the unsharded job.

    ``dist`` is ``torch.distributed`` (or None for a single process); ``rollout_factory`` builds
    the per-rank driver and exists so that the layout and gather logic can be exercised on
    machines without a GPU.
    """

    def __init__(self, total_groups: int, n_expand: int, elems: int, n_steps: int,
                 stages: Sequence[Tuple[int, int]], seed: int, vel_dtype: torch.dtype,
                 adv_eps: float = 1e-6, logp_mean: bool = False, dist=None, group=None,
                 rollout_factory: Optional[Callable] = None):
        self.dist = dist if (dist is not None and dist.is_initialized()) else None
        self.group = group
        self.rank = self.dist.get_rank(group) if self.dist else 0
        self.world = self.dist.get_world_size(group) if self.dist else 1
        self.total_groups, self.n_expand = total_groups, n_expand
        self.final_keep = stages[-1][1] if len(stages) else n_expand
        self.shards = [sharding.group_shard(total_groups, self.world, r) for r in range(self.world)]
        self.first, self.count = self.shards[self.rank]
        factory = rollout_factory or _default_factory
        self.local = None
        if self.count > 0:
            self.local = factory(self.count, n_expand, elems, n_steps, stages, seed, vel_dtype,
                                 adv_eps=adv_eps, group_offset=self.first, logp_mean=logp_mean)

    @property
    def local_rows(self) -> slice:
        """Rows of this rank's trajectories in an array laid out over the whole job's G_total * N0
        initial trajectories."""
        return slice(self.first * self.n_expand, (self.first + self.count) * self.n_expand)

    def run(self, x0_local, step_coef, preview_coef, velocity, **kw):
        """Runs this rank's shard (``Rollout.run`` arguments; x0_local holds the shard's rows
        only).  Returns the local ``RolloutOutput``, or None on a rank without groups."""
        if self.local is None:
            return None
        return self.local.run(x0_local, step_coef, preview_coef, velocity, **kw)

    def max_over_ranks(self, value: float, device=None) -> float:
        return sharding.max_over_ranks(value, self.dist, device)

    def gather(self, out, device=None) -> GatheredResults:
        """All-gathers the per-group results of every rank's ``run`` output in global group order.
        Collective: every rank of the group must call it (ranks without groups pass None)."""
        k = self.final_keep
        if out is None:
            dev = device or "cpu"
            empty_f = torch.empty(0, dtype=torch.float32, device=dev)
            adv = rewards = mean = std = empty_f
            ids = torch.empty(0, dtype=torch.int32, device=dev)
        else:
            adv, rewards, mean, std, ids = (out.adv.reshape(-1), out.rewards.reshape(-1),
                                            out.mean.reshape(-1), out.std.reshape(-1),
                                            out.traj_id.reshape(-1))
            assert adv.shape[0] == self.count * k and mean.shape[0] == self.count
        g = lambda t: sharding.all_gather_groups(t, self.dist, self.group)
        return GatheredResults(adv=g(adv), rewards=g(rewards), mean=g(mean), std=g(std), traj_id=g(ids),
                               shards=list(self.shards))

    def close(self):
        if self.local is not None:
            self.local.close()
            self.local = None


# ------------------------------------------------------------------ launcher

def _group_velocity(w, step: int, first: int, count: int, device) -> torch.Tensor:
    """Stand-in predictions of the groups [first, first + count) at `step`, drawn group by group
    from generators keyed by (seed, step, global group), so that any sharding of the job feeds
    every group the same bytes."""
    from . import workloads as wl
    per = w.rows_before(step)
    out = torch.empty(count * per, w.elems, device=device,
                      dtype=torch.bfloat16 if w.vel_dtype == "bf16" else torch.float32)
    for j in range(count):
        g = wl._gen(device, w.seed, 404, step, first + j)
        out[j * per:(j + 1) * per] = torch.randn(per, w.elems, generator=g, device=device,
                                                 dtype=torch.float32).to(out.dtype)
    return out


def main(argv=None) -> int:
    from . import binding as B
    from . import workloads as wl
    from .rollout import initial_latents
    ap = argparse.ArgumentParser(description="group-sharded Expand-and-Prune rollout, one rank per GPU")
    ap.add_argument("--workload", default="sd3",
                    choices=[n for n, w in wl.WORKLOADS.items() if w.velocity == "normal"],
                    help="shape and schedule; scores are the preview mean for every workload here")
    ap.add_argument("--groups", type=int, default=0, help="prompt groups of the whole job (default: the workload's)")
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args(argv)
    import torch.distributed as dist
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    launched = "RANK" in os.environ and "WORLD_SIZE" in os.environ
    if launched:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()
    from dataclasses import replace
    w = replace(wl.WORKLOADS[args.workload], scores="preview")
    total = args.groups or w.n_groups
    dt = torch.bfloat16 if w.vel_dtype == "bf16" else torch.float32
    sr = ShardedRollout(total, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, dt, adv_eps=w.adv_eps,
                        dist=dist if launched else None)
    x0 = vels = None
    if sr.count:
        x0 = initial_latents(w.seed, sr.count, w.n_expand, w.elems, group_offset=sr.first, device=dev)
        vels = [_group_velocity(w, s, sr.first, sr.count, dev) for s in range(w.n_steps)]
    run = lambda: sr.run(x0, w.step_coef, w.preview_coef, lambda s, x: vels[s])
    for _ in range(3):
        out = run()
    torch.cuda.synchronize()
    if launched:
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.reps):
        out = run()
    b.record()
    torch.cuda.synchronize()
    ms = sr.max_over_ranks(a.elapsed_time(b) / args.reps, dev)
    res = sr.gather(out, device=dev)
    whole = replace(w, n_groups=total)
    if sr.rank == 0:
        print(json.dumps({
            "workload": w.name, "groups": total, "ranks": sr.world, "shards": res.shards,
            "ms_per_rollout_max_over_ranks": ms,
            "latent_steps_per_s": whole.traj_steps / (ms * 1e-3),
            "survivors": int(res.traj_id.numel()),
            "adv_abs_mean_per_group_max": float(res.adv.view(total, -1).mean(dim=1).abs().max()),
            "adv_checksum": float(res.adv.double().abs().sum()),
            "traj_id_checksum": int(res.traj_id.long().sum()),
            "collectives": "all-gather of adv / rewards / mean / std / traj_id after the rollout; none inside it"}))
    sr.close()
    if launched:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
