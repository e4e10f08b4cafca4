"""Pins for the oracle's clustering diagnostics and uniform-subsampling baseline."""
import math

import numpy as np
import pytest
from scipy import stats

import oracle
from paper_2512_15347_b200 import workloads as wl


def test_group_stats_hand_case_and_numpy():
    # {0,0,0,0,10}: mean 2, variance (4*4 + 64)/5 = 16, sigma 4; delta 0.5 -> |R-2| <= 2: the zeros
    sc = np.array([[0, 0, 0, 0, 10]], np.float32)
    mean, std, frac = oracle.group_stats(sc, 0.5)
    assert (mean[0], std[0], frac[0]) == (2.0, 4.0, 0.8)
    assert oracle.group_stats(sc, 0.49)[2][0] == 0.0
    assert oracle.group_stats(sc, 2.0)[2][0] == 1.0
    rng = np.random.default_rng(0)
    r = rng.standard_normal((6, 40)).astype(np.float32)
    mean, std, _ = oracle.group_stats(r, 1.0)
    np.testing.assert_allclose(mean, r.astype(np.float64).mean(1), rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(std, r.astype(np.float64).std(1), rtol=1e-13)
    # normal scores: P(|z| <= delta) = erf(delta / sqrt 2)
    big = rng.standard_normal((1, 200000)).astype(np.float32)
    for delta in (0.5, 1.0, 2.0):
        frac = oracle.group_stats(big, delta)[2][0]
        assert frac == pytest.approx(math.erf(delta / math.sqrt(2)), abs=5e-3)
    # constant group: sigma 0, everything is inside
    assert oracle.group_stats(np.full((1, 7), 3.0, np.float32), 0.1)[2][0] == 1.0


def test_clustered_members_have_bounded_advantage():
    """Eq. adv-bound: members of C_delta have |A| <= delta."""
    sc = wl.clustered_scores(50, 24, 3, 0, cluster_sigma=0.05, outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
    mean, std, frac = oracle.group_stats(sc, 0.5)
    adv, _, _ = oracle.advantages(sc, 1e-6)
    inside = np.abs(sc.astype(np.float64) - mean[:, None]) <= 0.5 * std[:, None]
    np.testing.assert_allclose(inside.mean(axis=1), frac, rtol=1e-12)
    assert np.all(np.abs(adv[inside]) <= 0.5)
    # the reward-clustering workload is clustered: most members lie within half a sigma
    assert frac.mean() > 0.55


def test_uniform_selection_is_a_valid_uniform_subset():
    G, n, k = 4000, 24, 12
    keep = oracle.select_uniform(G, n, k, seed=11, stage=0)
    assert keep.shape == (G, k)
    assert np.all(np.diff(keep, axis=1) > 0) and keep.min() >= 0 and keep.max() < n
    counts = np.bincount(keep.reshape(-1), minlength=n)
    # every slot is kept with probability k/n
    chi2 = ((counts - G * k / n) ** 2 / (G * k / n * (1 - k / n))).sum()
    assert stats.chi2.sf(chi2, n - 1) > 1e-4
    # pairs of slots are kept together with probability k(k-1)/(n(n-1))
    together = np.mean([(0 in row) and (n - 1 in row) for row in keep.tolist()])
    assert together == pytest.approx(k * (k - 1) / (n * (n - 1)), abs=0.03)
    # stage, seed, group offset all change the draw; the draw itself is reproducible
    np.testing.assert_array_equal(keep, oracle.select_uniform(G, n, k, 11, 0))
    assert not np.array_equal(keep, oracle.select_uniform(G, n, k, 11, 1))
    assert not np.array_equal(keep, oracle.select_uniform(G, n, k, 12, 0))
    np.testing.assert_array_equal(keep[5:9], oracle.select_uniform(4, n, k, 11, 0, group_offset=5))
    np.testing.assert_array_equal(oracle.select_uniform(3, 7, 7, 1, 0), np.tile(np.arange(7), (3, 1)))


def test_uniform_subsampling_does_not_raise_variance_but_ovf_does():
    """Section 4.1: a uniform subset keeps the clustering (E[var] = var_full * n(k-1) / ((n-1)k)),
    OVF spreads it."""
    G, n, k = 3000, 24, 12
    sc = wl.clustered_scores(G, n, 9, 0, cluster_sigma=0.05, outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
    full = sc.astype(np.float64).var(axis=1)
    uni = oracle.select_uniform(G, n, k, 5, 0)
    var_uni = np.take_along_axis(sc, uni, axis=1).astype(np.float64).var(axis=1)
    expect = full.mean() * n * (k - 1) / ((n - 1) * k)
    assert var_uni.mean() == pytest.approx(expect, rel=0.1)
    _, var_ovf = oracle.ovf_select(sc, k)
    assert var_ovf.mean() > 1.5 * var_uni.mean()
