"""The N > 1 path on CPU: two gloo ranks each run their shard of the groups (through the oracle,
with the global group offset) and together reproduce the unsharded rollout; timing reduction
takes the maximum over ranks."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, total_groups, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2512_15347_b200 import sharding, workloads as wl
        w = wl.scaled(wl.WORKLOADS["sd15"], n_groups=total_groups, elems=64)
        first, count = sharding.group_shard(total_groups, world, rank)
        x0 = wl.initial_latents(w).numpy()
        rows = slice(first * w.n_expand, (first + count) * w.n_expand)

        def vel(s, x, traj):
            per = w.rows_before(s)
            full = wl.as_numpy_velocity(wl.normal_velocity(w, s, total_groups * per))
            return full[first * per:(first + count) * per]

        res = oracle.rollout(x0[rows], count, w.n_expand, w.n_steps, w.stages, w.seed, w.step_coef,
                             w.preview_coef, vel, adv_eps=w.adv_eps, group_offset=first)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), x=res.x_final, adv=res.adv,
                 ids=res.traj_id, keep=res.stage_keep[0], logp=np.concatenate(res.logp))
        # timing reduction: every rank must see the slowest rank's time
        slowest = sharding.max_over_ranks(10.0 + rank, dist)
        assert slowest == 10.0 + world - 1
        # equal shards gather back into global group order
        mine = torch.full((2, 3), float(rank))
        whole = sharding.all_gather_groups(mine, dist)
        assert whole.shape == (2 * world, 3)
        assert torch.equal(whole[:, 0], torch.arange(world).repeat_interleave(2).float())
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_rollout(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2512_15347_b200 import sharding, workloads as wl
    total, world = 5, 2
    port = 29500 + (os.getpid() % 2000)
    mp.start_processes(_worker, args=(world, port, total, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    w = wl.scaled(wl.WORKLOADS["sd15"], n_groups=total, elems=64)
    x0 = wl.initial_latents(w).numpy()
    ref = oracle.rollout(x0, total, w.n_expand, w.n_steps, w.stages, w.seed, w.step_coef, w.preview_coef,
                         lambda s, x, traj: wl.as_numpy_velocity(
                             wl.normal_velocity(w, s, total * w.rows_before(s))),
                         adv_eps=w.adv_eps)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    np.testing.assert_array_equal(np.concatenate([p["x"] for p in parts]), ref.x_final)
    np.testing.assert_array_equal(np.concatenate([p["ids"] for p in parts]), ref.traj_id)
    np.testing.assert_array_equal(np.concatenate([p["keep"] for p in parts]), ref.stage_keep[0])
    np.testing.assert_array_equal(np.concatenate([p["adv"] for p in parts]), ref.adv)
    # shards tile the groups without gaps or overlap
    spans = [sharding.group_shard(total, world, r) for r in range(world)]
    assert spans == [(0, 3), (3, 2)]
    assert sharding.weak_shard(64, 3) == (192, 64)
    with pytest.raises(ValueError):
        sharding.group_shard(4, 2, 2)
