"""GPU parity of the policy-update calls (log-prob of stored transitions + KL, clipped
surrogate objective, gradient w.r.t. the prediction) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_15347_b200 import workloads as wl
from tests import util as U

pytestmark = pytest.mark.gpu


def grad_err(a, b) -> float:
    """max_e |a-b| / max(|b_e|, rms(b_row))"""
    return U.latent_err(a, b)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("d", [4, 1000, 3 * 8192 + 20, 65536])
@pytest.mark.parametrize("logp_mean", [False, True])
def test_policy_update_matches_oracle(bf16, d, logp_mean):
    from paper_2512_15347_b200 import binding as B
    G, K, T = 3, 4, 3
    n = G * K
    rng = np.random.default_rng(d + 7 * bf16 + logp_mean)
    coef = (1.0, 0.1, 0.25)
    vd = B.VEL_BF16 if bf16 else B.VEL_F32
    h = B.rollout_init(B.make_config(G, K, d, T, [], 3, vd, logp_mean=logp_mean))

    def vel(arr):
        t = torch.from_numpy(arr.astype(np.float32))
        return wl.as_numpy_velocity(t.to(torch.bfloat16) if bf16 else t)

    try:
        xs = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(T)]
        v_old = [vel(rng.standard_normal((n, d))) for _ in range(T)]
        # new prediction close to the old one so that ratios stay finite in sum mode
        delta = 2e-3 if not logp_mean else 0.5
        v_new, xn = [], []
        for t in range(T):
            vo = U.vel_to_dev(v_old[t]).float().cpu().numpy()
            v_new.append(vel(vo + delta * rng.standard_normal((n, d))))
            xn.append((xs[t] + coef[1] * vo + coef[2] * rng.standard_normal((n, d))).astype(np.float32))
        adv = rng.standard_normal(n).astype(np.float32)
        lp_old = np.stack([oracle.policy_logprob(xs[t], xn[t], v_old[t], None, *coef, logp_mean)[0]
                           for t in range(T)]).astype(np.float32)

        lp_new = torch.empty(T, n, device="cuda")
        kl = torch.empty(T, n, device="cuda")
        dev = [(U.to_dev(xs[t]), U.to_dev(xn[t]), U.vel_to_dev(v_new[t]), U.vel_to_dev(v_old[t]))
               for t in range(T)]
        ref_lp, ref_kl = [], []
        for t in range(T):
            B.policy_logprob(h, coef, dev[t][0], dev[t][1], dev[t][2], dev[t][3], lp_new[t], kl[t])
            a, b = oracle.policy_logprob(xs[t], xn[t], v_new[t], v_old[t], *coef, logp_mean)
            ref_lp.append(a)
            ref_kl.append(b)
        scale = 1.0 if logp_mean else d
        got_lp = lp_new.cpu().numpy()
        assert (np.abs(got_lp - np.stack(ref_lp)) / np.maximum(np.abs(np.stack(ref_lp)), 0.5 * scale)).max() <= 1e-5
        np.testing.assert_allclose(kl.cpu().numpy(), np.stack(ref_kl), rtol=1e-5, atol=1e-30)
        # without a reference the log-prob is unchanged
        lp_only = torch.empty(n, device="cuda")
        B.policy_logprob(h, coef, dev[0][0], dev[0][1], dev[0][2], None, lp_only, None)
        assert torch.equal(lp_only, lp_new[0])

        # objective from the device's own fp32 log-probs
        ratio = torch.empty(T, n, device="cuda")
        dlogp = torch.empty(T, n, device="cuda")
        obj = torch.empty(1, device="cuda")
        B.policy_objective(h, T, lp_new, U.to_dev(lp_old), kl, U.to_dev(adv), 0.2, 0.3, ratio, dlogp, obj)
        ref_obj, ref_ratio, ref_dlogp = oracle.policy_objective(got_lp, lp_old, kl.cpu().numpy(), adv, 0.2, 0.3)
        np.testing.assert_allclose(ratio.cpu().numpy(), ref_ratio, rtol=1e-6)
        np.testing.assert_allclose(dlogp.cpu().numpy(), ref_dlogp, rtol=1e-6, atol=1e-30)
        assert float(obj.item()) == pytest.approx(ref_obj, rel=1e-5, abs=1e-7)

        # gradient for every step
        dkl = -0.3 / (T * n)
        for t in range(T):
            g = torch.empty(n, d, device="cuda", dtype=torch.bfloat16 if bf16 else torch.float32)
            B.policy_backward(h, coef, dev[t][0], dev[t][1], dev[t][2], dev[t][3], dlogp[t], dkl, g)
            ref_g = oracle.policy_backward(xs[t], xn[t], v_new[t], v_old[t], *coef,
                                           dlogp[t].cpu().numpy().astype(np.float64), dkl, logp_mean)
            tol = 2.0 ** -8 if bf16 else 1e-5
            assert grad_err(g.float().cpu().numpy(), ref_g) <= tol
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_policy_update_after_a_rollout_has_unit_ratio():
    """Re-evaluating the rollout's own predictions gives back its log-probs: ratio 1, objective =
    mean advantage = 0, and the objective's gradient is A / (nT) * dlogp/dv."""
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.Workload("upd", 4, 8, (), 3, 8192 + 512, 1, "bf16", 5, "normal", "preview")
    inp = U.SharedInputs(w)
    ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16, logp_mean=True)
    xs = [U.to_dev(inp.x0)]
    vels = []

    def velocity(s, x):
        v = inp.vel_device(s, x)
        vels.append(v)
        if s > 0:
            xs.append(x.clone())
        return v

    out = ro.run(xs[0], w.step_coef, w.preview_coef, velocity)
    xs.append(out.x_final.clone())
    n, T = w.n_groups * w.n_expand, w.n_steps
    lp_new = torch.empty(T, n, device="cuda")
    for t in range(T):
        B.policy_logprob(ro.h, w.step_coef(t), xs[t], xs[t + 1], vels[t], None, lp_new[t], None)
    lp_old = torch.stack(out.logp)
    torch.cuda.synchronize()
    # fp32 storage of x_{t+1} perturbs the recomputed mean log-prob by ~1e-7
    assert (lp_new - lp_old).abs().max().item() < 2e-6
    ratio = torch.empty(T, n, device="cuda")
    dlogp = torch.empty(T, n, device="cuda")
    obj = torch.empty(1, device="cuda")
    B.policy_objective(ro.h, T, lp_new, lp_old, None, out.adv, 0.2, 0.0, ratio, dlogp, obj)
    torch.cuda.synchronize()
    assert (ratio - 1).abs().max().item() < 1e-5
    assert abs(obj.item()) < 1e-6
    ro.close()


def test_unit_ratio_in_sum_mode_on_full_length_latents():
    """Summed log-densities (the form of Eq. ratio_method) on 16x128x128 latents: pg_step reports
    log pi from the generator's radius terms, pg_policy_logprob recomputes it from the stored fp32
    x_{t+1}; the two differ by the fp32 rounding of x_{t+1} and of the noise transform, an error
    that grows with the latent length.  Bound asserted (and documented in the header):
    |log pi_new - log pi_old| <= 2e-6 * d, the mean-mode bound times d."""
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.Workload("upd-sum", 2, 3, (), 3, 262144, 1, "bf16", 9, "normal", "preview")
    inp = U.SharedInputs(w)
    ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16, logp_mean=False)
    xs = [U.to_dev(inp.x0)]
    vels = []

    def velocity(s, x):
        v = inp.vel_device(s, x)
        vels.append(v)
        if s > 0:
            xs.append(x.clone())
        return v

    out = ro.run(xs[0], w.step_coef, w.preview_coef, velocity)
    xs.append(out.x_final.clone())
    n, T, d = w.n_groups * w.n_expand, w.n_steps, w.elems
    lp_new = torch.empty(T, n, device="cuda")
    for t in range(T):
        B.policy_logprob(ro.h, w.step_coef(t), xs[t], xs[t + 1], vels[t], None, lp_new[t], None)
    lp_old = torch.stack(out.logp)
    torch.cuda.synchronize()
    gap = (lp_new.double() - lp_old.double()).abs().max().item()
    print(f"sum-mode |log pi_new - log pi_old| max {gap:.4f} at d = {d} ({gap / d:.2e} per element)")
    assert gap <= 2e-6 * d
    # the oracle's density of the stored transition agrees with the recomputed value to fp32 accuracy
    ref = oracle.policy_logprob(xs[0].cpu().numpy(), xs[1].cpu().numpy(), wl.as_numpy_velocity(vels[0]), None,
                                *w.step_coef(0), False)[0]
    assert U.logp_err(lp_new[0].cpu().numpy(), ref, d) <= U.LOGP_TOL
    ro.close()


def test_objective_over_many_entries_matches_oracle():
    """T * n = 50 x 8192 entries: the objective kernel runs as 50 CTAs whose partial sums are
    combined in slot order; same result on every run, and the oracle's within fp32 rounding."""
    from paper_2512_15347_b200 import binding as B
    T, G, K = 50, 1024, 8
    n = G * K
    rng = np.random.default_rng(77)
    h = B.rollout_init(B.make_config(G, K, 4, T, [], 1, B.VEL_F32, logp_mean=True))
    try:
        lp_old = rng.standard_normal((T, n)).astype(np.float32)
        lp_new = (lp_old + 0.3 * rng.standard_normal((T, n))).astype(np.float32)
        kl = (0.1 * rng.random((T, n))).astype(np.float32)
        adv = rng.standard_normal(n).astype(np.float32)
        outs = []
        for _ in range(3):
            ratio = torch.empty(T, n, device="cuda")
            dlogp = torch.empty(T, n, device="cuda")
            obj = torch.full((1,), float("nan"), device="cuda")
            B.policy_objective(h, T, U.to_dev(lp_new), U.to_dev(lp_old), U.to_dev(kl), U.to_dev(adv), 0.2, 0.04,
                               ratio, dlogp, obj)
            torch.cuda.synchronize()
            outs.append((obj.clone(), ratio, dlogp))
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[1][0], outs[2][0])
        ref_obj, ref_ratio, ref_dlogp = oracle.policy_objective(lp_new, lp_old, kl, adv, 0.2, 0.04)
        assert float(outs[0][0].item()) == pytest.approx(ref_obj, rel=2e-6, abs=1e-9)
        np.testing.assert_allclose(outs[0][1].cpu().numpy(), ref_ratio, rtol=1e-6)
        np.testing.assert_allclose(outs[0][2].cpu().numpy(), ref_dlogp, rtol=1e-6, atol=1e-30)
        # a number of entries that is not a multiple of anything, and one that fits a single CTA
        for t_small, n_rows in ((7, 3001), (1, 5)):
            hs = B.rollout_init(B.make_config(n_rows, 1, 4, t_small, [], 1, B.VEL_F32, logp_mean=True))
            a, b = lp_new.reshape(-1)[: t_small * n_rows].reshape(t_small, n_rows), lp_old.reshape(-1)[: t_small * n_rows].reshape(t_small, n_rows)
            ad = adv[:n_rows]
            dl = torch.empty(t_small, n_rows, device="cuda")
            ob = torch.empty(1, device="cuda")
            B.policy_objective(hs, t_small, U.to_dev(a), U.to_dev(b), None, U.to_dev(ad), 0.1, 0.0, None, dl, ob)
            torch.cuda.synchronize()
            r_obj, _, r_dl = oracle.policy_objective(a, b, None, ad, 0.1, 0.0)
            assert float(ob.item()) == pytest.approx(r_obj, rel=2e-6, abs=1e-9)
            np.testing.assert_allclose(dl.cpu().numpy(), r_dl, rtol=1e-6, atol=1e-30)
            B.rollout_destroy(hs)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_policy_update_on_the_survivors_of_a_pruned_rollout():
    """The whole chain after a rollout with two prunes: the survivors' transitions are collected
    from the stored steps (rows from pg_survivor_rows, latents and predictions through
    pg_gather_rows), re-evaluated under the same predictions, and give back the survivors' own
    log-prob history (pg_survivor_logp): ratio 1 at every step, objective = mean advantage = 0."""
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.Workload("upd-pruned", 3, 12, ((1, 6), (3, 2)), 5, 8192 + 512, 1, "bf16", 9, "normal", "preview")
    inp = U.SharedInputs(w)
    ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16, logp_mean=True)
    xs, vels = [], []

    def velocity(s, x):
        v = inp.vel_device(s, x)
        xs.append(x.clone())                   # x_s in the layout of the rows alive before any prune at s
        vels.append(v)
        return v

    out = ro.run(U.to_dev(inp.x0), w.step_coef, w.preview_coef, velocity)
    xs.append(out.x_final.clone())
    T, n = w.n_steps, w.n_groups * w.final_keep
    rows = torch.empty(T, n, dtype=torch.int32, device="cuda")
    B.survivor_rows(ro.h, torch.cat(out.stage_keep), rows)
    lp_old = torch.empty(T, n, device="cuda")
    B.survivor_logp(ro.h, rows, torch.cat(out.logp), lp_old)
    orig = (out.traj_id - 0).to(torch.int32)   # group_offset 0: the original row of every survivor
    lp_new = torch.empty(T, n, device="cuda")
    d = w.elems
    for t in range(T):
        rows_in = orig if t == 0 else rows[t - 1]
        n_in = xs[t].shape[0]
        x_t = torch.empty(n, d, device="cuda")
        v_t = torch.empty(n, d, device="cuda", dtype=torch.bfloat16)
        B.gather_rows(ro.h, rows_in, n, n_in, xs[t], x_t, d * 4)
        B.gather_rows(ro.h, rows_in, n, n_in, vels[t], v_t, d * 2)
        if t + 1 < T:
            x_n = torch.empty(n, d, device="cuda")
            B.gather_rows(ro.h, rows[t], n, xs[t + 1].shape[0], xs[t + 1], x_n, d * 4)
        else:
            x_n = xs[T]
        B.policy_logprob(ro.h, w.step_coef(t), x_t, x_n, v_t, None, lp_new[t], None)
    torch.cuda.synchronize()
    assert B.rollout_status(ro.h)[2] == 0
    assert (lp_new - lp_old).abs().max().item() < 2e-6
    ratio = torch.empty(T, n, device="cuda")
    dlogp = torch.empty(T, n, device="cuda")
    obj = torch.empty(1, device="cuda")
    B.policy_objective(ro.h, T, lp_new, lp_old, None, out.adv, 0.2, 0.0, ratio, dlogp, obj)
    torch.cuda.synchronize()
    assert (ratio - 1).abs().max().item() < 1e-5
    assert abs(obj.item()) < 1e-6
    ro.close()
