"""Coefficient builders against the mathematics they encode: for Gaussian data the exact network
prediction is linear, so a correct sampler must reproduce the data distribution (the SDE
conversions of Section 3.2 are meant to leave the marginal distributions unchanged)."""
import math

import numpy as np
import pytest

import oracle
from paper_2512_15347_b200 import binding as B
from paper_2512_15347_b200 import schedules as S

MU, SD = 1.5, 0.4          # 1-D Gaussian data N(MU, SD^2), replicated over independent elements
N, D = 4000, 4


def _integrate(coefs, predict, x):
    ids = np.arange(N, dtype=np.int32)
    for s, coef in enumerate(coefs):
        pred = predict(s, x.astype(np.float64)).astype(np.float32)
        x, _ = oracle.step(x, pred, ids, 123, s, *coef)
    return x.astype(np.float64)


def _check_data_distribution(x, tol_mean=0.03, tol_sd=0.05):
    assert abs(x.mean() - MU) < tol_mean
    assert x.std() == pytest.approx(SD, rel=tol_sd)


def _rf_velocity(t, x):
    # E[x_1 - x_0 | x_t] for x_t = (1 - t) x_0 + t x_1
    var = (1 - t) ** 2 + (t * SD) ** 2
    return MU + (t * SD * SD - (1 - t)) / var * (x - t * MU)


@pytest.mark.parametrize("sigma", [0.0, 0.7, 1.2])
def test_rf_sde_keeps_the_marginals(sigma):
    T = 400
    rng = np.random.default_rng(0)
    x0 = rng.standard_normal((N, D)).astype(np.float32)
    ts = S.uniform_times(T)
    coefs = [S.rf_sde_coef(t, 1.0 / T, sigma) for t in ts]
    x = _integrate(coefs, lambda s, x: _rf_velocity(ts[s], x), x0)
    _check_data_distribution(x)
    # the sign of the score term matters: the opposite sign inflates the spread
    if sigma > 0:
        wrong = [(2.0 - c[0], 2.0 / T - c[1], c[2]) for c in coefs]
        xw = _integrate(wrong, lambda s, x: _rf_velocity(ts[s], x), x0)
        assert xw.std() > 1.5 * SD
    # halfway through, the latent follows the path's marginal N(t MU, (1-t)^2 + t^2 SD^2)
    xh = _integrate(coefs[: T // 2], lambda s, x: _rf_velocity(ts[s], x), x0)
    assert abs(xh.mean() - 0.5 * MU) < 0.03
    assert xh.std() == pytest.approx(math.sqrt(0.25 + 0.25 * SD * SD), rel=0.05)


def test_rf_drift_coef_and_preview():
    assert S.rf_drift_coef(0.1, 0.7) == (1.0, 0.1, 0.7 * math.sqrt(0.1))
    assert S.rf_sde_coef(0.3, 0.05, 0.0) == (1.0, 0.05, 0.0)
    # point-mass data: the one-step preview lands on the data point from any time
    for t in (0.0, 0.3, 0.9):
        x0 = np.linspace(-2, 2, 7)
        xt = (1 - t) * x0 + t * MU
        v = MU - x0
        p_x, p_v = S.rf_preview_coef(t)
        np.testing.assert_allclose(p_x * xt + p_v * v, MU, atol=1e-12)


def _eps_prediction(alpha, sigma, x):
    # E[eps | x_t] for x_t = alpha x_1 + sigma eps
    return sigma * (x - alpha * MU) / (alpha * alpha * SD * SD + sigma * sigma)


@pytest.mark.parametrize("eta", [0.0, 0.5, 1.0])
def test_ddim_schedule_reaches_the_data_distribution(eta):
    steps = 500            # few-step DDIM contracts the spread of Gaussian data (0.37 at 50 steps)
    alpha, sigma = S.vp_linear_schedule()
    ts = [round(999 * (1.0 - s / steps)) for s in range(steps)]
    rng = np.random.default_rng(1)
    x_T = (alpha[999] * (MU + SD * rng.standard_normal((N, D))) + sigma[999] * rng.standard_normal((N, D)))
    x = _integrate(S.ddim_schedule(steps, eta), lambda s, x: _eps_prediction(alpha[ts[s]], sigma[ts[s]], x),
                   x_T.astype(np.float32))
    _check_data_distribution(x)
    # eta = 0 is deterministic
    assert all(c[2] == 0.0 for c in S.ddim_schedule(steps, 0.0))
    assert all(c[2] > 0.0 for c in S.ddim_schedule(steps, 1.0)[:-1])
    # clean-sample preview is exact for point-mass data
    a, s = alpha[500], sigma[500]
    eps = np.linspace(-2, 2, 5)
    p_x, p_v = S.x0_preview_coef(a, s)
    np.testing.assert_allclose(p_x * (a * MU + s * eps) + p_v * eps, MU, atol=1e-12)


@pytest.mark.parametrize("eta", [0.0, 1.0])
def test_vp_euler_maruyama_keeps_the_marginals(eta):
    # continuous linear beta(t) on [0, 1]: alpha_bar = exp(-int beta / 2), integrate from t = 1 to 0
    T = 1000
    b0, b1 = 0.1, 12.0
    beta = lambda t: b0 + (b1 - b0) * t
    abar = lambda t: math.exp(-0.5 * (b0 * t + 0.5 * (b1 - b0) * t * t))
    ts = [1.0 - s / T for s in range(T)]
    rng = np.random.default_rng(2)
    a1 = abar(1.0)
    s1 = math.sqrt(1 - a1 * a1)
    x = (a1 * (MU + SD * rng.standard_normal((N, D))) + s1 * rng.standard_normal((N, D))).astype(np.float32)
    coefs = [S.vp_em_coef(beta(t), math.sqrt(1 - abar(t) ** 2), 1.0 / T, eta) for t in ts]
    x = _integrate(coefs, lambda s, x: _eps_prediction(abar(ts[s]), math.sqrt(1 - abar(ts[s]) ** 2), x), x)
    _check_data_distribution(x, tol_mean=0.04, tol_sd=0.08)
    p_x, p_v = S.vp_euler_preview_coef(2.0, 0.5, 0.25)
    assert (p_x, p_v) == (1.25, -0.5)


def test_paper_schedules_are_accepted():
    for name, (g_max, stages, T) in S.PAPER_SCHEDULES.items():
        S.validate_stages(g_max, T, stages)
        cfg = B.make_config(2, g_max, 64, T, stages, 0, B.VEL_BF16)
        assert B.rollout_host_workspace_bytes(cfg) > 0, name
    with pytest.raises(ValueError):
        S.validate_stages(8, 10, [(3, 9)])
    with pytest.raises(ValueError):
        S.validate_stages(8, 10, [(3, 4), (3, 2)])
    with pytest.raises(ValueError):
        S.rf_sde_coef(1.0, 0.1, 0.5)
