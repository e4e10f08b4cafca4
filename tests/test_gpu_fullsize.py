"""Full-size parity: the large workload exactly as bench.py launches it (64 groups x 64
trajectories, d = 262144, bf16 predictions generated on the device), checked against the oracle
on sampled prompt groups followed end to end, plus whole-batch properties."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_15347_b200 import workloads as wl
from tests import util as U

pytestmark = pytest.mark.gpu

SAMPLED_GROUPS = (0, 5, 17, 31, 37, 50, 62, 63)


def test_large_workload_sampled_groups_match_oracle():
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.WORKLOADS["large"]
    free, _ = torch.cuda.mem_get_info()
    if free < 24e9:
        pytest.skip("needs 24 GB of free device memory")
    dev = torch.device("cuda")
    ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16,
                 adv_eps=w.adv_eps)
    x0 = wl.initial_latents(w, device=dev)
    host_x0 = {g: x0[g * w.n_expand:(g + 1) * w.n_expand].cpu().numpy() for g in SAMPLED_GROUPS}
    host_vel = {g: [] for g in SAMPLED_GROUPS}

    def velocity(s, x_active):
        rows = w.n_groups * w.rows_before(s)
        v = wl.normal_velocity(w, s, rows, device=dev)
        per = w.rows_before(s)
        for g in SAMPLED_GROUPS:
            host_vel[g].append(wl.as_numpy_velocity(v[g * per:(g + 1) * per]))
        return v

    out = ro.run(x0, w.step_coef, w.preview_coef, velocity, record_scores=True)
    torch.cuda.synchronize()
    assert B.rollout_status(ro.h) == (w.n_groups * w.final_keep, w.n_steps, 0)

    # whole batch: the selection is the oracle's, bit for bit, on the device's own scores
    k_prev = w.n_expand
    for i, (s, k) in enumerate(w.stages):
        sc = out.stage_scores[i].cpu().numpy().reshape(w.n_groups, k_prev)
        keep = out.stage_keep[i].cpu().numpy().reshape(w.n_groups, k)
        np.testing.assert_array_equal(keep, oracle.ovf_select(sc, k)[0])
        assert np.all(np.diff(keep, axis=1) > 0)
        k_prev = k
    # third stage keeps everything
    np.testing.assert_array_equal(out.stage_keep[2].cpu().numpy().reshape(w.n_groups, 16),
                                  np.tile(np.arange(16), (w.n_groups, 1)))
    # whole batch: advantages of the device's rewards
    rw = out.rewards.cpu().numpy().reshape(w.n_groups, w.final_keep)
    ref_adv, ref_mean, ref_std = oracle.advantages(rw, w.adv_eps)
    np.testing.assert_allclose(out.adv.cpu().numpy().reshape(rw.shape), ref_adv, rtol=1e-5, atol=1e-6)
    assert np.abs(out.adv.cpu().numpy().reshape(rw.shape).mean(axis=1)).max() < 1e-6
    # whole batch: E[log pi] = -(d/2)(1 + ln(2 pi s^2)) for every step
    for s in range(w.n_steps):
        ns = w.step_coef(s)[2]
        want = -0.5 * w.elems * (1 + np.log(2 * np.pi * ns * ns))
        lp = out.logp[s].cpu().numpy().astype(np.float64)
        assert abs(lp.mean() - want) < 6 * np.sqrt(w.elems / 2) / np.sqrt(lp.size)

    # sampled groups: the oracle follows each group through the whole schedule
    k_final = w.final_keep
    for g in SAMPLED_GROUPS:
        ref = oracle.rollout(host_x0[g], 1, w.n_expand, w.n_steps, w.stages, w.seed, w.step_coef,
                             w.preview_coef, lambda s, x, traj, g=g: host_vel[g][s],
                             adv_eps=w.adv_eps, group_offset=g)
        k_prev = w.n_expand
        for i, (s, k) in enumerate(w.stages):
            got_sc = out.stage_scores[i].cpu().numpy().reshape(w.n_groups, k_prev)[g]
            assert np.abs(got_sc.astype(np.float64) - ref.stage_scores[i][0]).max() <= U.SCORE_GAP
            np.testing.assert_array_equal(out.stage_keep[i].cpu().numpy().reshape(w.n_groups, k)[g],
                                          ref.stage_keep[i][0])
            k_prev = k
        for s in range(w.n_steps):
            per = w.active_at(s)
            got = out.logp[s].cpu().numpy()[g * per:(g + 1) * per]
            assert U.logp_err(got, ref.logp[s], w.elems) <= U.LOGP_TOL
        got_x = out.x_final[g * k_final:(g + 1) * k_final].cpu().numpy()
        assert U.latent_err(got_x, ref.x_final) <= U.LATENT_TOL
        np.testing.assert_array_equal(out.traj_id.cpu().numpy()[g * k_final:(g + 1) * k_final],
                                      ref.traj_id)
        np.testing.assert_allclose(out.adv.cpu().numpy().reshape(w.n_groups, k_final)[g], ref.adv[0],
                                   rtol=2e-4, atol=2e-5)
    ro.close()


def test_ovf_microbench_shape_matches_oracle():
    """The selection microbenchmark's exact workload: 4096 groups x 256 scores -> 32."""
    from paper_2512_15347_b200 import binding as B
    m = wl.OVF_MICRO
    sc = wl.ovf_micro_scores()
    G, n, k = m["n_groups"], m["n"], m["k"]
    keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
    kept = torch.empty(G * k, device="cuda")
    adv = torch.empty(G * k, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ovf_select_batched(G, n, k, U.to_dev(sc), keep, kept, adv, 1e-6, st)
    ref_keep, _ = oracle.ovf_select(sc, k)
    np.testing.assert_array_equal(keep.cpu().numpy().reshape(G, k), ref_keep)
    ref_kept = np.take_along_axis(sc, ref_keep, axis=1)
    np.testing.assert_array_equal(kept.cpu().numpy().reshape(G, k), ref_kept)
    ref_adv, _, _ = oracle.advantages(ref_kept, 1e-6)
    np.testing.assert_allclose(adv.cpu().numpy().reshape(G, k), ref_adv, rtol=1e-5, atol=1e-6)
    assert int(st.item()) == 0


def test_sd3_workload_full_size_matches_oracle_everywhere():
    """The SD3 / FLUX-shaped workload (16 groups x 48 -> 24 -> 12, 28 steps, 16x128x128 latents,
    external clustered scores) is small enough for the oracle to follow every trajectory."""
    from paper_2512_15347_b200 import binding as B
    w = wl.WORKLOADS["sd3"]
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    ro, out = U.run_gpu(w, inp)
    lp_err, x_err = U.compare_rollouts(w, ref, out)
    assert B.rollout_status(ro.h) == (w.n_groups * w.final_keep, w.n_steps, 0)
    # selection statistics the method is about: the kept subset is more spread out than the group
    for i, (s, k) in enumerate(w.stages):
        sc = ref.stage_scores[i].astype(np.float64)
        assert np.all(ref.stage_var[i] >= sc.var(axis=1) - 1e-12)
    ro.close()
