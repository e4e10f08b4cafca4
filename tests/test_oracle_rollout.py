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


def test_survivor_rows_hand_cases():
    # one group of 4, pruned to slots {1, 3} before step 1 of 3
    rows = oracle.survivor_rows(1, 4, 3, [(1, 2)], [np.array([[1, 3]])])
    assert rows.tolist() == [[1, 3], [0, 1], [0, 1]]
    # two groups of 5: 5 -> 3 before step 0 (slots differ per group), 3 -> 1 before step 2
    keep0 = np.array([[0, 2, 4], [1, 2, 3]])
    keep1 = np.array([[2], [0]])
    rows = oracle.survivor_rows(2, 5, 4, [(0, 3), (2, 1)], [keep0, keep1])
    # group 0 survivor: original slot 4, row 2 of its 3 rows; group 1 survivor: original slot 1, row 0
    assert rows.tolist() == [[2, 3 + 0], [2, 3 + 0], [0, 1], [0, 1]]
    # no stages: identity at every step
    assert oracle.survivor_rows(2, 3, 2, [], []).tolist() == [list(range(6))] * 2


def test_survivor_rows_point_at_the_survivors_own_transitions():
    """Pinned by the noise: row rows[t][j] of step t's latents is the trajectory whose id the j-th
    final survivor carries, so its transition x_{t+1} - (x_t + dt v_t) is noise_std times that
    trajectory's own normals of step t (generator keyed by trajectory id), and no other row's."""
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=3, elems=64)
    x0 = wl.initial_latents(w).numpy()
    vels = [wl.as_numpy_velocity(wl.normal_velocity(w, s, w.n_groups * w.rows_before(s))) for s in range(w.n_steps)]
    res = oracle.rollout(x0, w.n_groups, w.n_expand, w.n_steps, w.stages, w.seed, w.step_coef, w.preview_coef,
                         lambda s, x, traj: vels[s], adv_eps=w.adv_eps, keep_steps=True, group_offset=2)
    rows = oracle.survivor_rows(w.n_groups, w.n_expand, w.n_steps, w.stages, res.stage_keep)
    n_final = w.n_groups * w.final_keep
    assert rows.shape == (w.n_steps, n_final)
    assert rows[-1].tolist() == list(range(n_final))            # after the last prune: dense, in order
    xs = [x0] + res.x_steps
    for t in range(w.n_steps):
        c_x, c_v, ns = w.step_coef(t)
        assert len(set(rows[t].tolist())) == n_final and rows[t].max() < w.n_groups * w.active_at(t)
        for j in (0, n_final // 2, n_final - 1):
            tid = int(res.traj_id[j])
            # x_t and its prediction are laid out as the rows alive after step t-1 (before any prune
            # scheduled at t): the survivor's row of the previous step, or its original slot at t = 0
            r_in = int(rows[t - 1][j]) if t > 0 else tid - 2 * w.n_expand
            x_t = xs[t][r_in].astype(np.float64)
            v_t = vels[t][r_in]
            v_t = (v_t.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
            x_n = xs[t + 1][int(rows[t][j])].astype(np.float64)
            xi = oracle.normal_row(w.seed, t, tid, w.elems)
            np.testing.assert_allclose(x_n - (c_x * x_t + c_v * v_t), ns * xi, atol=2e-6)
    # the survivors' log-prob history, picked out of the packed per-step arrays
    lp = np.stack([res.logp[t][rows[t]] for t in range(w.n_steps)])
    assert lp.shape == (w.n_steps, n_final) and np.isfinite(lp).all()
