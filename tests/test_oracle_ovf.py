"""Pins for the oracle's Optimal Variance Filtering, compaction and advantages:
brute force over all subsets, hand-worked cases, numpy statistics, invariants."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2512_15347_b200 import workloads as wl


def _hand_cases(golden_dir):
    for line in open(os.path.join(golden_dir, "ovf_hand_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        sc, k, keep, var = [p.strip() for p in line.split("|")]
        yield (np.array(sc.split(), dtype=np.float32), int(k),
               [int(t) for t in keep.split()], Fraction(var))


def test_hand_cases(golden_dir):
    cases = list(_hand_cases(golden_dir))
    assert len(cases) == 6
    for scores, k, keep, var in cases:
        got_keep, got_var = oracle.ovf_select(scores, k)
        assert list(got_keep) == keep
        assert got_var[0] == pytest.approx(float(var), rel=1e-14, abs=1e-300)
        ex_var, _ = oracle.ovf_exhaustive(scores, k)
        assert ex_var == pytest.approx(float(var), rel=1e-14, abs=1e-300)


def test_exhaustive_search_is_numpy_brute_force():
    rng = np.random.default_rng(3)
    for n, k in [(5, 2), (6, 3), (7, 5), (8, 4), (4, 4), (5, 1)]:
        sc = rng.standard_normal(n).astype(np.float32)
        want = max(np.var(sc[list(c)].astype(np.float64)) for c in itertools.combinations(range(n), k))
        got, subset = oracle.ovf_exhaustive(sc, k)
        assert got == pytest.approx(want, rel=1e-13, abs=1e-300)
        assert np.var(sc[subset].astype(np.float64)) == pytest.approx(want, rel=1e-13, abs=1e-300)


def _instances():
    rng = np.random.default_rng(12345)
    for trial in range(600):
        n = int(rng.integers(2, 13))
        k = int(rng.integers(1, n + 1))
        kind = trial % 5
        if kind == 0:
            sc = rng.standard_normal(n)
        elif kind == 1:
            sc = rng.integers(0, 3, n).astype(np.float64)          # heavy ties
        elif kind == 2:
            sc = rng.standard_t(1.5, n)                              # heavy tails
        elif kind == 3:
            sc = 1000.0 + 1e-3 * rng.standard_normal(n)             # large offset, tiny spread
        else:
            sc = np.where(rng.random(n) < 0.2, 0.3 * rng.standard_t(3, n),
                          0.05 * rng.standard_normal(n)) + rng.random()
        yield sc.astype(np.float32), k


def test_scan_reaches_the_exhaustive_optimum():
    """The 'j lowest + k-j highest' scan attains the maximum of Eq. ovf: heuristic gap 0."""
    worst = 0.0
    for sc, k in _instances():
        ex_var, _ = oracle.ovf_exhaustive(sc, k)
        keep, var = oracle.ovf_select(sc, k)
        assert len(set(keep.tolist())) == k and list(keep) == sorted(keep)
        direct = np.var(sc[keep].astype(np.float64))
        scale = max(ex_var, 1e-300)
        # pivot-centred sums lose at most a few ulp of the largest squared deviation
        tol = 1e-12 * scale + 1e-13 * float(np.max(np.abs(sc.astype(np.float64) - np.median(sc))) ** 2)
        assert abs(var[0] - direct) <= tol
        assert abs(direct - ex_var) <= tol
        worst = max(worst, (ex_var - direct) / scale)
    assert worst <= 1e-12


@pytest.mark.parametrize("n,k", [(16, 8), (24, 12), (24, 16), (16, 12), (48, 24), (48, 32), (32, 8),
                                 (64, 8), (64, 32), (256, 32), (16, 16), (100, 1), (100, 99)])
def test_local_optimality_on_paper_shapes(n, k):
    """No single in/out exchange raises the variance (necessary for the argmax of Eq. ovf)."""
    sc = wl.clustered_scores(3, n, seed=n * 131 + k, stage=0, cluster_sigma=0.05,
                             outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
    keep, var = oracle.ovf_select(sc, k)
    for g in range(sc.shape[0]):
        r = sc[g].astype(np.float64)
        inside = keep[g].tolist()
        assert inside == sorted(set(inside)) and len(inside) == k
        base = np.var(r[inside])
        assert var[g] == pytest.approx(base, rel=1e-10, abs=1e-300)
        outside = [i for i in range(n) if i not in set(inside)]
        for i in inside:
            for o in outside:
                trial = [o if t == i else t for t in inside]
                assert np.var(r[trial]) <= base * (1 + 1e-12) + 1e-300


def test_ties_and_degenerate_sizes():
    same = np.full(9, 2.5, np.float32)
    np.testing.assert_array_equal(oracle.ovf_select(same, 4)[0], [0, 1, 2, 3])
    sc = np.array([3, 1, 4, 1, 5, 9, 2, 6], np.float32)
    np.testing.assert_array_equal(oracle.ovf_select(sc, 8)[0], np.arange(8))
    # k = 1: zero variance for every choice, the rule keeps the lowest (score, slot)
    np.testing.assert_array_equal(oracle.ovf_select(sc, 1)[0], [1])
    # -0 and +0 are the same score: the slot decides
    z = np.array([0.0, -0.0, 1.0, -1.0], np.float32)
    np.testing.assert_array_equal(oracle.ovf_select(z, 3)[0], [0, 2, 3])
    with pytest.raises(ValueError):
        oracle.ovf_select(sc, 9)
    with pytest.raises(ValueError):
        oracle.ovf_select(sc, 0)


def test_non_finite_scores_still_give_a_valid_subset():
    sc = np.array([0.1, np.nan, -np.inf, 0.3, np.inf, 0.2, 0.25, np.nan], np.float32)
    for k in range(1, 9):
        keep, var = oracle.ovf_select(sc, k)
        assert list(keep) == sorted(set(keep.tolist())) and len(keep) == k
        assert np.isfinite(var[0])
    # NaN orders above +inf, -inf lowest: with k = 2 the extremes are -inf and the last NaN
    np.testing.assert_array_equal(oracle.ovf_select(sc, 2)[0], [2, 7])


def test_ovf_raises_spread_over_uniform_subsampling():
    """Section 4.2 / Fig. 2a: the OVF subset has a larger standard deviation than the full
    group and than a uniformly drawn subset of the same size."""
    sc = wl.clustered_scores(200, 24, seed=5, stage=0, cluster_sigma=0.05, outlier_frac=0.15,
                             outlier_scale=0.3, nu=3.0)
    keep, var = oracle.ovf_select(sc, 12)
    rng = np.random.default_rng(0)
    full = sc.astype(np.float64).std(axis=1)
    uni = np.array([sc[g, rng.choice(24, 12, replace=False)].astype(np.float64).std()
                    for g in range(200)])
    assert np.all(np.sqrt(var) >= full - 1e-12)
    assert np.sqrt(var).mean() > 1.2 * full.mean() > 1.1 * uni.mean() * 0.9
    assert np.mean(np.sqrt(var) >= uni) == 1.0


def test_compaction_preserves_order_count_and_bytes():
    g, n, k, d = 5, 12, 7, 9
    rng = np.random.default_rng(8)
    sc = rng.standard_normal((g, n)).astype(np.float32)
    keep, _ = oracle.ovf_select(sc, k)
    rows = rng.standard_normal((g * n, d)).astype(np.float32)
    out = oracle.compact_rows(keep, rows, n)
    assert out.shape == (g * k, d)
    for gi in range(g):
        assert np.all(np.diff(keep[gi]) > 0)
        np.testing.assert_array_equal(out[gi * k:(gi + 1) * k], rows[gi * n + keep[gi]])
    ids = np.arange(g * n, dtype=np.int32).reshape(-1, 1)
    id1 = oracle.compact_rows(keep, ids, n).reshape(-1)
    assert np.all(np.diff(id1.reshape(g, k), axis=1) > 0)
    # two stages compose: ids after the second stage index the original rows directly
    sc2 = rng.standard_normal((g, k)).astype(np.float32)
    keep2, _ = oracle.ovf_select(sc2, 3)
    id2 = oracle.compact_rows(keep2, id1.reshape(-1, 1), k).reshape(-1)
    rows2 = oracle.compact_rows(keep2, out, k)
    np.testing.assert_array_equal(rows2, rows[id2])
    bad = keep.copy()
    bad[0, 0] = n
    with pytest.raises(ValueError):
        oracle.compact_rows(bad, rows, n)


def test_advantages_against_numpy_and_invariants():
    rng = np.random.default_rng(2)
    r = rng.standard_normal((7, 12)).astype(np.float32) * 3 + 1
    eps = 1e-6
    adv, mean, std = oracle.advantages(r, eps)
    r64 = r.astype(np.float64)
    np.testing.assert_allclose(mean, r64.mean(axis=1), rtol=1e-13)
    np.testing.assert_allclose(std, r64.std(axis=1, ddof=0), rtol=1e-13)
    np.testing.assert_allclose(adv, (r64 - r64.mean(1, keepdims=True)) / (r64.std(1, keepdims=True) + eps),
                               rtol=1e-12, atol=1e-15)
    assert np.abs(adv.mean(axis=1)).max() < 1e-12
    np.testing.assert_allclose(adv.std(axis=1), std / (std + eps), rtol=1e-12)
    # population, not sample, standard deviation
    assert not np.allclose(std, r64.std(axis=1, ddof=1))
    # invariance under R -> a R + b (a > 0), up to eps
    adv2, _, _ = oracle.advantages((2.0 * r + 5.0).astype(np.float32), eps)
    np.testing.assert_allclose(adv2, adv, atol=1e-5)
    # constant group: sigma = 0, advantages 0
    adv3, _, std3 = oracle.advantages(np.full((1, 6), 4.0, np.float32), eps)
    assert std3[0] == 0.0 and np.all(adv3 == 0.0)
    # clustered members are bounded: |R - mu| <= delta sigma  =>  |A| <= delta (Eq. adv-bound)
    for delta in (0.25, 0.5, 1.0):
        near = np.abs(r64 - mean[:, None]) <= delta * std[:, None]
        assert np.all(np.abs(adv[near]) <= delta)
