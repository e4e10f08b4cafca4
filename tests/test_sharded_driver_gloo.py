"""ShardedRollout on CPU: gloo ranks with unequal shards (and a rank without any group) run their
blocks of prompt groups through a stand-in per-rank driver built on the oracle, and the gathered
per-group results equal the unsharded rollout in global group order on every rank."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleRollout:
    """Per-rank driver with the constructor and run() signature of rollout.Rollout, computing with
    the CPU oracle (test stand-in: the product's driver needs a GPU)."""

    def __init__(self, n_groups, n_expand, elems, n_steps, stages, seed, vel_dtype, adv_eps=1e-6,
                 group_offset=0, logp_mean=False):
        self.args = (n_groups, n_expand, n_steps, stages, seed)
        self.adv_eps, self.group_offset = adv_eps, group_offset

    def run(self, x0, step_coef, preview_coef, velocity, **kw):
        import oracle
        from types import SimpleNamespace
        n_groups, n_expand, n_steps, stages, seed = self.args
        r = oracle.rollout(x0, n_groups, n_expand, n_steps, stages, seed, step_coef, preview_coef,
                           lambda s, x, traj: velocity(s, x), adv_eps=self.adv_eps,
                           group_offset=self.group_offset)
        t = torch.from_numpy
        return SimpleNamespace(adv=t(r.adv.astype(np.float32)), rewards=t(r.rewards), mean=t(r.mean.astype(np.float32)),
                               std=t(r.std.astype(np.float32)), traj_id=t(r.traj_id))

    def close(self):
        pass


def _workload(total):
    from paper_2512_15347_b200 import workloads as wl
    return wl.scaled(wl.WORKLOADS["sd15"], n_groups=total, elems=64)


def _velocity(w, total, first, count):
    from paper_2512_15347_b200 import workloads as wl

    def vel(s, x):
        per = w.rows_before(s)
        full = wl.as_numpy_velocity(wl.normal_velocity(w, s, total * per))
        return full[first * per:(first + count) * per]
    return vel


def _worker(rank, world, port, total, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2512_15347_b200 import workloads as wl
        from paper_2512_15347_b200.sharded import ShardedRollout
        w = _workload(total)
        sr = ShardedRollout(total, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16,
                            adv_eps=w.adv_eps, dist=dist, rollout_factory=OracleRollout)
        assert (sr.rank, sr.world) == (rank, world)
        assert sum(c for _, c in sr.shards) == total and sr.shards[rank] == (sr.first, sr.count)
        x0 = wl.initial_latents(w).numpy()[sr.local_rows]
        out = sr.run(x0, w.step_coef, w.preview_coef, _velocity(w, total, sr.first, sr.count))
        assert (out is None) == (sr.count == 0)
        res = sr.gather(out)
        slowest = sr.max_over_ranks(5.0 + rank)
        assert slowest == 5.0 + world - 1
        # one rank failing a local step makes every rank skip what follows, together
        from paper_2512_15347_b200 import sharding
        assert sharding.all_ranks_ok(True, dist) is True
        assert sharding.all_ranks_ok(rank != world - 1, dist) is False
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), adv=res.adv.numpy(), rewards=res.rewards.numpy(),
                 mean=res.mean.numpy(), std=res.std.numpy(), ids=res.traj_id.numpy(),
                 shards=np.array(res.shards))
        sr.close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("total,world", [(5, 2), (2, 3)])
def test_gathered_results_equal_the_unsharded_rollout(tmp_path, total, world):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2512_15347_b200 import workloads as wl
    port = 31500 + (os.getpid() % 2000) + world
    mp.start_processes(_worker, args=(world, port, total, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    w = _workload(total)
    ref = oracle.rollout(wl.initial_latents(w).numpy(), total, w.n_expand, w.n_steps, w.stages, w.seed,
                         w.step_coef, w.preview_coef, lambda s, x, traj: _velocity(w, total, 0, total)(s, x),
                         adv_eps=w.adv_eps)
    for r in range(world):
        got = np.load(tmp_path / f"rank{r}.npz")
        np.testing.assert_array_equal(got["ids"], ref.traj_id)
        np.testing.assert_array_equal(got["rewards"], ref.rewards.reshape(-1))
        np.testing.assert_array_equal(got["adv"], ref.adv.astype(np.float32).reshape(-1))
        np.testing.assert_array_equal(got["mean"], ref.mean.astype(np.float32))
        np.testing.assert_array_equal(got["std"], ref.std.astype(np.float32))
        assert got["shards"][:, 1].sum() == total
    if (total, world) == (2, 3):
        assert np.load(tmp_path / "rank2.npz")["shards"].tolist() == [[0, 1], [1, 1], [2, 0]]


def test_single_process_needs_no_process_group():
    from paper_2512_15347_b200.sharded import ShardedRollout
    w = _workload(3)
    sr = ShardedRollout(3, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16,
                        rollout_factory=OracleRollout)
    assert (sr.rank, sr.world, sr.first, sr.count) == (0, 1, 0, 3)
    from paper_2512_15347_b200 import workloads as wl
    out = sr.run(wl.initial_latents(w).numpy(), w.step_coef, w.preview_coef, _velocity(w, 3, 0, 3))
    res = sr.gather(out)
    assert res.adv.shape == (3 * w.final_keep,) and res.shards == [(0, 3)]
    assert float(res.adv.view(3, -1).mean(dim=1).abs().max()) < 1e-6
