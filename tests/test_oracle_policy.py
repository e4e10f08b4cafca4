"""Pins for the oracle's policy-update arithmetic (Eq. ratio_method, Eq. pro_grpo_method):
scipy densities, numerically integrated KL, hand-worked clipping cases, finite differences."""
import math

import numpy as np
import pytest
from scipy import integrate, stats

import oracle


def _data(n=3, d=8, seed=0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d)).astype(np.float32)
    v = rng.standard_normal((n, d)).astype(np.float32)
    vref = (v + 0.1 * rng.standard_normal((n, d))).astype(np.float32)
    xn = (x + 0.1 * v + 0.2 * rng.standard_normal((n, d))).astype(np.float32)
    return x, xn, v, vref


def test_logprob_is_scipy_density_and_step_logp_is_recovered():
    x, xn, v, vref = _data()
    c_x, c_v, s = 0.97, 0.1, 0.2
    lp, kl = oracle.policy_logprob(x, xn, v, vref, c_x, c_v, s)
    mean = c_x * x.astype(np.float64) + c_v * v.astype(np.float64)
    for i in range(x.shape[0]):
        want = stats.multivariate_normal.logpdf(xn[i].astype(np.float64), mean=mean[i], cov=s * s * np.eye(x.shape[1]))
        assert lp[i] == pytest.approx(want, rel=1e-12)
    lp_mean, kl_mean = oracle.policy_logprob(x, xn, v, vref, c_x, c_v, s, logp_mean=True)
    np.testing.assert_allclose(lp_mean, lp / x.shape[1], rtol=1e-14)
    np.testing.assert_allclose(kl_mean, kl / x.shape[1], rtol=1e-14)
    # the same prediction as in the rollout gives back the rollout's log-prob (ratio 1)
    ids = np.arange(3, dtype=np.int32)
    x_next, lp_roll = oracle.step(x, v, ids, 5, 2, c_x, c_v, s)
    lp_again, _ = oracle.policy_logprob(x, x_next, v, None, c_x, c_v, s)
    np.testing.assert_allclose(lp_again, lp_roll, rtol=0, atol=2e-4)   # fp32 storage of x_next


def test_kl_against_numerical_integration():
    # d = 1: KL(N(m1, s^2) || N(m2, s^2)) = integral p1 (log p1 - log p2)
    x = np.array([[0.5]], np.float32)
    v = np.array([[1.25]], np.float32)
    vref = np.array([[-0.75]], np.float32)
    c_x, c_v, s = 1.0, 0.3, 0.4
    _, kl = oracle.policy_logprob(x, x, v, vref, c_x, c_v, s)
    m1, m2 = 0.5 + 0.3 * 1.25, 0.5 - 0.3 * 0.75
    f = lambda t: stats.norm.pdf(t, m1, s) * (stats.norm.logpdf(t, m1, s) - stats.norm.logpdf(t, m2, s))
    want, _ = integrate.quad(f, m1 - 12 * s, m1 + 12 * s, epsabs=1e-13, epsrel=1e-13)
    assert kl[0] == pytest.approx(want, rel=1e-9)
    # d > 1: independent coordinates add up; and KL(p || p) = 0
    x4, xn4, v4, vref4 = _data(2, 4, 3)
    _, kl4 = oracle.policy_logprob(x4, xn4, v4, vref4, c_x, c_v, s)
    per = sum(oracle.policy_logprob(x4[:, e:e + 1], xn4[:, e:e + 1], v4[:, e:e + 1], vref4[:, e:e + 1], c_x, c_v, s)[1]
              for e in range(4))
    np.testing.assert_allclose(kl4, per, rtol=1e-13)
    _, kl0 = oracle.policy_logprob(x4, xn4, v4, v4, c_x, c_v, s)
    assert np.all(kl0 == 0.0)


def test_clipped_surrogate_hand_cases():
    # T = 1, four trajectories, eps = 0.2: ratios 1.5, 1.5, 0.5, 1.1 with advantages +2, -2, +2, -1
    lr = np.log(np.array([[1.5, 1.5, 0.5, 1.1]]))
    adv = np.array([2.0, -2.0, 2.0, -1.0])
    obj, ratio, dlogp = oracle.policy_objective(lr, np.zeros((1, 4)), None, adv, 0.2, 0.0)
    np.testing.assert_allclose(ratio[0], [1.5, 1.5, 0.5, 1.1], rtol=1e-15)
    # min(3, 2.4) = 2.4 (clipped); min(-3, -2.4) = -3; min(1, 1.6) = 1; min(-1.1, -1.1) = -1.1
    assert obj == pytest.approx((2.4 - 3.0 + 1.0 - 1.1) / 4, rel=1e-14)
    # gradient flows only where the unclipped branch is active: d(rA)/dlogp = rA
    np.testing.assert_allclose(dlogp[0], np.array([0.0, -3.0, 1.0, -1.1]) / 4, rtol=1e-14)
    # KL term: J decreases by beta * mean(kl)
    kl = np.array([[0.1, 0.2, 0.3, 0.4]])
    obj2, _, _ = oracle.policy_objective(lr, np.zeros((1, 4)), kl, adv, 0.2, 0.5)
    assert obj2 == pytest.approx(obj - 0.5 * 0.25, rel=1e-14)
    # ratio 1 everywhere: J = mean advantage (0 for group-normalised advantages)
    obj3, r3, d3 = oracle.policy_objective(np.ones((3, 4)), np.ones((3, 4)), None, adv, 0.2, 0.0)
    assert obj3 == pytest.approx(adv.mean(), rel=1e-14) and np.all(r3 == 1.0)
    np.testing.assert_allclose(d3, np.tile(adv, (3, 1)) / 12, rtol=1e-14)


@pytest.mark.parametrize("logp_mean", [False, True])
def test_backward_matches_finite_differences(logp_mean):
    n, d, T = 4, 6, 2
    rng = np.random.default_rng(7)
    c_x, c_v, s, eps, beta = 1.0, 0.2, 0.5, 0.2, 0.3
    xs = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(T)]
    vs = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(T)]
    vrefs = [(v + 0.3 * rng.standard_normal((n, d))).astype(np.float32) for v in vs]
    xns = [(x + c_v * v + s * rng.standard_normal((n, d))).astype(np.float32) for x, v in zip(xs, vs)]
    adv = rng.standard_normal(n)
    lp_old = np.stack([oracle.policy_logprob(xs[t], xns[t], vrefs[t], None, c_x, c_v, s, logp_mean)[0]
                       for t in range(T)])

    def J(vels):
        lp, kl = zip(*[oracle.policy_logprob(xs[t], xns[t], vels[t], vrefs[t], c_x, c_v, s, logp_mean)
                       for t in range(T)])
        return oracle.policy_objective(np.stack(lp), lp_old, np.stack(kl), adv, eps, beta)

    obj, ratio, dlogp = J(vs)
    if not logp_mean:
        assert (ratio < 1 - eps).any() or (ratio > 1 + eps).any()  # some entries are clipped
    grads = [oracle.policy_backward(xs[t], xns[t], vs[t], vrefs[t], c_x, c_v, s, dlogp[t],
                                    -beta / (n * T), logp_mean) for t in range(T)]
    h = 2.0 ** -7                                                  # exact in fp32 next to O(1) values
    for t, i, e in [(0, 0, 0), (0, 3, 5), (1, 1, 2), (1, 2, 4), (0, 2, 1), (1, 0, 3)]:
        plus = [v.copy() for v in vs]
        minus = [v.copy() for v in vs]
        plus[t][i, e] += h
        minus[t][i, e] -= h
        step = float(plus[t][i, e]) - float(minus[t][i, e])
        fd = (J(plus)[0] - J(minus)[0]) / step
        assert grads[t][i, e] == pytest.approx(fd, rel=2e-3, abs=1e-7)
