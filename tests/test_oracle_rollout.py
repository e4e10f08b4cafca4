"""Oracle-level checks of the whole Expand-and-Prune rollout (schedule semantics)."""
import numpy as np

import oracle
from paper_2512_15347_b200 import workloads as wl
from tests import util as U


def test_schedule_counts_and_id_composition():
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=2, elems=64)
    inp = U.SharedInputs(w)
    res = U.run_oracle(w, inp)
    assert [len(lp) for lp in res.logp] == [2 * w.active_at(s) for s in range(w.n_steps)]
    assert sum(len(lp) for lp in res.logp) == w.traj_steps
    # ids after all stages = original ids indexed stage after stage
    ids = np.arange(2 * w.n_expand).reshape(2, -1)
    for keep in res.stage_keep:
        ids = np.take_along_axis(ids, keep, axis=1)
    np.testing.assert_array_equal(res.traj_id, ids.reshape(-1))
    # the degenerate third stage (keep == active) is the identity
    np.testing.assert_array_equal(res.stage_keep[2], np.tile(np.arange(16), (2, 1)))
    # survivors' advantages: zero mean, unit population std (up to eps)
    assert np.abs(res.adv.mean(axis=1)).max() < 1e-9
    np.testing.assert_allclose(res.adv.std(axis=1), res.std / (res.std + w.adv_eps), rtol=1e-9)


def test_pruned_trajectories_do_not_influence_survivors():
    """A survivor's latent equals the one obtained by running that trajectory alone."""
    w = wl.scaled(wl.WORKLOADS["sd15"], n_groups=1, elems=32)
    inp = U.SharedInputs(w)
    res = U.run_oracle(w, inp)
    tid = int(res.traj_id[0])
    x = inp.x0[tid:tid + 1]
    for s in range(w.n_steps):
        v = inp.vel_numpy(s, np.empty((w.n_groups * w.rows_before(s), 0)))
        # the row this trajectory occupies when step s is predicted
        if s <= w.stages[0][0]:
            row = tid
        else:
            row = int(np.where(res.stage_keep[0][0] == tid)[0][0])
        x, _ = oracle.step(x, v[row:row + 1], np.array([tid], np.int32), w.seed, s, *w.step_coef(s))
    np.testing.assert_array_equal(x[0], res.x_final[0])


def test_resume_reproduces_the_run():
    w = wl.scaled(wl.WORKLOADS["tiny"], elems=64)
    inp = U.SharedInputs(w)
    res = U.run_oracle(w, inp, keep_steps=True)
    # restart after step 5 (post-prune) from the stored latent
    x = res.x_steps[5]
    ids = res.traj_id
    a, b = inp.affine
    for s in range(6, w.n_steps):
        v = inp.vel_numpy(s, x)
        x, _ = oracle.step(x, v, ids, w.seed, s, *w.step_coef(s))
    np.testing.assert_array_equal(x, res.x_final)
