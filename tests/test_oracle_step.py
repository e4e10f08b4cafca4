"""Pins for the oracle's SDE step, Gaussian log-probability and preview score:
closed forms, scipy's normal density, moment recursions of the Euler-Maruyama chain."""
import math

import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from paper_2512_15347_b200 import workloads as wl


def _rand(n, d, seed=0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, d)).astype(np.float32)


def test_deterministic_limit_is_exact():
    x = _rand(3, 16)
    v = _rand(3, 16, 1)
    ids = np.arange(3, dtype=np.int32)
    out, lp = oracle.step(x, v, ids, seed=1, step_index=0, c_x=0.5, c_v=0.0, noise_std=0.0)
    np.testing.assert_array_equal(out, 0.5 * x)
    np.testing.assert_array_equal(lp, 0.0)
    out, _ = oracle.step(x, v, ids, seed=1, step_index=0, c_x=1.0, c_v=0.25, noise_std=0.0)
    want = (x.astype(np.float64) + 0.25 * v.astype(np.float64)).astype(np.float32)
    np.testing.assert_array_equal(out, want)


def test_update_adds_scaled_generator_noise():
    n, d, seed, s = 4, 64, 9, 3
    x, v = _rand(n, d), _rand(n, d, 1)
    ids = np.array([7, 3, 11, 0], dtype=np.int32)
    c_x, c_v, ns = 1.0, 0.1, 0.7 * math.sqrt(0.1)
    out, _ = oracle.step(x, v, ids, seed, s, c_x, c_v, ns)
    for i in range(n):
        xi = oracle.normal_row(seed, s, int(ids[i]), d)
        want = c_x * x[i].astype(np.float64) + c_v * v[i].astype(np.float64) + ns * xi
        np.testing.assert_allclose(out[i], want, rtol=0, atol=1e-6)
        # and the residual really is N(0, ns^2): the sign and the scale are right
        resid = (out[i] - (x[i] + c_v * v[i])) / ns
        assert np.corrcoef(resid, xi)[0, 1] > 0.999999


def test_logp_is_the_gaussian_density_scipy():
    n, d = 3, 8
    x, v = _rand(n, d, 2), _rand(n, d, 3)
    x_next = np.random.default_rng(4).standard_normal((n, d))
    c_x, c_v, ns = 0.9, 0.2, 0.3
    got = oracle.transition_logp(x, v, x_next, c_x, c_v, ns)
    mean = c_x * x.astype(np.float64) + c_v * v.astype(np.float64)
    for i in range(n):
        want = stats.multivariate_normal.logpdf(x_next[i], mean=mean[i], cov=ns * ns * np.eye(d))
        assert got[i] == pytest.approx(want, rel=1e-12)
    got_mean = oracle.transition_logp(x, v, x_next, c_x, c_v, ns, logp_mean=True)
    np.testing.assert_allclose(got_mean, got / d, rtol=1e-14)


def test_logp_hand_values_d1_d2():
    # d = 1: x=0, v=0 -> mean 0; x' = 1, std 2: log N(1; 0, 4) = -1/8 - ln(2) - ln(2 pi)/2
    x = np.zeros((1, 1), np.float32)
    got = oracle.transition_logp(x, x, np.array([[1.0]]), 1.0, 1.0, 2.0)
    assert got[0] == pytest.approx(-0.125 - math.log(2.0) - 0.5 * math.log(2 * math.pi), rel=1e-14)
    # d = 2: mean (1, -1) from x=(2,-2), c_x=.5; x' = (1.5, -1), std .5:
    #   -1/2 * ((.5/.5)^2 + 0) - ln(2 pi * .25)
    x = np.array([[2.0, -2.0]], np.float32)
    got = oracle.transition_logp(x, x, np.array([[1.5, -1.0]]), 0.5, 0.0, 0.5)
    assert got[0] == pytest.approx(-0.5 - math.log(2 * math.pi * 0.25), rel=1e-14)


def test_step_logp_equals_density_of_its_own_sample():
    """Sampling-mode identity: log pi = -1/2 sum xi^2 - d/2 ln(2 pi s^2), and the value
    reported by step() is the density of the latent it produced."""
    n, d, seed, s = 5, 256, 21, 2
    x, v = _rand(n, d, 5), _rand(n, d, 6)
    ids = np.arange(10, 10 + n, dtype=np.int32)
    c_x, c_v, ns = 1.0, 0.05, 0.2
    out, lp = oracle.step(x, v, ids, seed, s, c_x, c_v, ns)
    for i in range(n):
        xi = oracle.normal_row(seed, s, int(ids[i]), d)
        want = -0.5 * np.sum(xi * xi) - 0.5 * d * math.log(2 * math.pi * ns * ns)
        assert lp[i] == pytest.approx(want, rel=1e-12)
    # density of the stored (fp32-rounded) sample agrees up to the storage rounding
    dens = oracle.transition_logp(x, v, out.astype(np.float64), c_x, c_v, ns)
    np.testing.assert_allclose(dens, lp, rtol=0, atol=1e-3)
    lp_mean = oracle.step(x, v, ids, seed, s, c_x, c_v, ns, logp_mean=True)[1]
    np.testing.assert_allclose(lp_mean, lp / d, rtol=1e-14)


def test_logp_population_mean():
    # E[log pi] = -(d/2) (1 + ln(2 pi s^2)), standard deviation sqrt(d/2) per trajectory
    n, d, ns = 256, 1024, 0.3
    x = np.zeros((n, d), np.float32)
    _, lp = oracle.step(x, x, np.arange(n, dtype=np.int32), 5, 0, 1.0, 0.0, ns)
    want = -0.5 * d * (1 + math.log(2 * math.pi * ns * ns))
    assert abs(lp.mean() - want) < 5 * math.sqrt(d / 2) / math.sqrt(n)
    assert lp.std() == pytest.approx(math.sqrt(d / 2), rel=0.25)


def test_gather_and_trajectory_ids():
    """Row i reads row src_slot[i]; noise follows the trajectory id, not the row position."""
    n, d = 6, 32
    x, v = _rand(n, d, 7), _rand(n, d, 8)
    ids = np.arange(n, dtype=np.int32) + 100
    full, lp_full = oracle.step(x, v, ids, 2, 4, 1.0, 0.1, 0.2)
    src = np.array([1, 4, 5], dtype=np.int32)
    part, lp_part = oracle.step(x, v, ids[src], 2, 4, 1.0, 0.1, 0.2, src_slot=src)
    np.testing.assert_array_equal(part, full[src])
    np.testing.assert_array_equal(lp_part, lp_full[src])


def test_bf16_velocity_decoding():
    x = np.zeros((1, 4), np.float32)
    bits = np.array([[0x3F80, 0xC000, 0x0000, 0x3DCD]], dtype=np.uint16)   # 1, -2, 0, 0.10009765625
    out, _ = oracle.step(x, bits, np.zeros(1, np.int32), 0, 0, 1.0, 1.0, 0.0)
    np.testing.assert_array_equal(out[0], np.array([1.0, -2.0, 0.0, 0.10009765625], np.float32))
    t = torch.tensor([[1.0, -2.0, 0.0, 0.1]]).to(torch.bfloat16)
    np.testing.assert_array_equal(wl.bf16_bits(t), bits)


def test_affine_field_moment_recursion():
    """Config-1 style chain v = a x + b: E[x_{s+1}] = (1 + a dt) E[x_s] + b dt and
    Var_{s+1} = (1 + a dt)^2 Var_s + noise_std^2, per channel."""
    w = wl.WORKLOADS["tiny"]
    n = 64
    a, b = wl.affine_field(w)
    x = torch.randn(n, w.elems, generator=torch.Generator().manual_seed(1)).numpy()
    ids = np.arange(n, dtype=np.int32)
    per = w.elems // w.channels
    mean = np.array([x[:, c * per:(c + 1) * per].mean() for c in range(w.channels)])
    var = np.array([x[:, c * per:(c + 1) * per].var() for c in range(w.channels)])
    a_c, b_c = a.numpy()[::per].astype(np.float64), b.numpy()[::per].astype(np.float64)
    for s in range(w.n_steps):
        c_x, c_v, ns = w.step_coef(s)
        v = wl.affine_velocity(torch.from_numpy(x), a, b).numpy()
        x, _ = oracle.step(x, v, ids, w.seed, s, c_x, c_v, ns)
        mean = (1 + a_c * c_v) * mean + b_c * c_v
        var = (1 + a_c * c_v) ** 2 * var + ns * ns
    m = n * per
    for c in range(w.channels):
        blk = x[:, c * per:(c + 1) * per].astype(np.float64)
        assert abs(blk.mean() - mean[c]) < 5 * math.sqrt(var[c] / m)
        assert blk.var() == pytest.approx(var[c], rel=5 * math.sqrt(2.0 / m))


def test_score_closed_forms():
    n, d = 4, 128
    x, v = _rand(n, d, 9), _rand(n, d, 10)
    zero = np.zeros_like(v)
    s0, _ = oracle.score(x, zero, 1.0, 0.37)
    np.testing.assert_allclose(s0, x.astype(np.float64).mean(axis=1), rtol=1e-13, atol=1e-16)
    const = np.full((n, d), 0.75, np.float32)
    s1, _ = oracle.score(const, v, 2.0, -0.5)
    np.testing.assert_allclose(s1, 1.5 - 0.5 * v.astype(np.float64).mean(axis=1), rtol=1e-12)
    # linear in (p_x, p_v)
    sa, _ = oracle.score(x, v, 1.0, 0.0)
    sb, _ = oracle.score(x, v, 0.0, 1.0)
    sc, prev = oracle.score(x, v, 0.3, 0.9, want_preview=True)
    np.testing.assert_allclose(sc, 0.3 * sa + 0.9 * sb, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(prev, 0.3 * x.astype(np.float64) + 0.9 * v.astype(np.float64),
                               rtol=1e-6)
    # x and v are not interchangeable
    sd, _ = oracle.score(v, x, 0.3, 0.9)
    assert not np.allclose(sc, sd)
