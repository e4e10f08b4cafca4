"""Pins for the oracle's counter-based noise: published Philox known answers and the
statistics / invertibility of the 24-bit Box-Muller transform."""
import os

import numpy as np
import pytest
from scipy import stats

import oracle


def _kat(golden_dir):
    rows = []
    for line in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert list(oracle.philox4x32_10(ctr, key)) == want


def test_philox_batch_matches_single():
    rng = np.random.default_rng(0)
    ctr = rng.integers(0, 2**32, size=(64, 4), dtype=np.uint64).astype(np.uint32)
    key = rng.integers(0, 2**32, size=(64, 2), dtype=np.uint64).astype(np.uint32)
    out = oracle.philox_batch(ctr, key)
    for i in range(64):
        assert tuple(out[i]) == oracle.philox4x32_10(ctr[i], key[i])


def test_philox_word_roles_are_distinct():
    # a transposed counter word or key word changes the block
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    assert oracle.philox4x32_10([2, 1, 3, 4], [5, 6]) != base
    assert oracle.philox4x32_10([1, 2, 4, 3], [5, 6]) != base
    assert oracle.philox4x32_10([1, 2, 3, 4], [6, 5]) != base


def test_normals_are_standard_normal():
    d = 1 << 18
    xi = np.concatenate([oracle.normal_row(11, s, t, d) for s in range(2) for t in range(2)])
    n = xi.size
    assert abs(xi.mean()) < 5.0 / np.sqrt(n)
    assert abs(xi.var() - 1.0) < 5.0 * np.sqrt(2.0 / n)
    assert abs(stats.kurtosis(xi)) < 5.0 * np.sqrt(24.0 / n)
    assert abs(stats.skew(xi)) < 5.0 * np.sqrt(6.0 / n)
    assert stats.kstest(xi, "norm").pvalue > 1e-3
    assert np.abs(xi).max() <= np.sqrt(2 * 24 * np.log(2.0)) + 1e-12   # u1 >= 2^-24
    # the four members of a quad and neighbouring quads are uncorrelated
    q = xi.reshape(-1, 4)
    c = np.corrcoef(q.T)
    assert np.abs(c - np.eye(4)).max() < 5.0 / np.sqrt(q.shape[0])
    assert abs(np.corrcoef(xi[:-4], xi[4:])[0, 1]) < 5.0 / np.sqrt(n)


def test_box_muller_inverts_to_the_generator_words():
    """radius^2 = -2 ln u1 and angle = 2 pi u2 recover the 24-bit uniforms that the raw
    Philox words of counter (q, step, trajectory, stream), key (seed_lo, seed_hi) define."""
    seed, step, traj, d = (0x1234ABCD << 32) | 0x9876, 5, 77, 64
    xi = oracle.normal_row(seed, step, traj, d).reshape(-1, 2, 2)
    for q in range(d // 4):
        r = oracle.philox4x32_10([q, step, traj, 0], [seed & 0xFFFFFFFF, seed >> 32])
        for p in range(2):
            a, b = xi[q, p]
            u1 = np.exp(-(a * a + b * b) / 2.0)
            u2 = (np.arctan2(b, a) / (2 * np.pi)) % 1.0
            assert abs(u1 * 2**24 - ((r[2 * p] >> 8) + 1)) < 1e-6 * 2**24 * u1 + 1e-6
            want_u2 = (r[2 * p + 1] >> 8) / 2**24
            assert min(abs(u2 - want_u2), 1 - abs(u2 - want_u2)) < 1e-9


def test_noise_key_fields_all_matter():
    base = oracle.normal_row(3, 1, 2, 16)
    assert not np.allclose(base, oracle.normal_row(4, 1, 2, 16))
    assert not np.allclose(base, oracle.normal_row(3 + (1 << 32), 1, 2, 16))
    assert not np.allclose(base, oracle.normal_row(3, 2, 2, 16))
    assert not np.allclose(base, oracle.normal_row(3, 1, 3, 16))
    assert not np.allclose(base, oracle.normal_row(3, 1, 2, 16, stream=1))
    # element e of a longer row is the same number: the counter holds e // 4, not d
    np.testing.assert_array_equal(base, oracle.normal_row(3, 1, 2, 64)[:16])
    with pytest.raises(ValueError):
        oracle.normal_row(3, 1, 2, 6)
