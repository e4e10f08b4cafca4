"""The seeded input generators are reproducible and have the stated shapes and statistics."""
import numpy as np
import torch

from paper_2512_15347_b200 import workloads as wl


def test_generators_are_deterministic():
    w = wl.scaled(wl.WORKLOADS["sd15"], elems=256)
    a, b = wl.initial_latents(w), wl.initial_latents(w)
    assert torch.equal(a, b) and a.shape == (8 * 24, 256) and a.dtype == torch.float32
    v1, v2 = wl.normal_velocity(w, 3, 96), wl.normal_velocity(w, 3, 96)
    assert torch.equal(v1, v2) and v1.dtype == torch.bfloat16
    assert not torch.equal(v1, wl.normal_velocity(w, 4, 96))
    s1 = wl.clustered_scores(4, 48, 3, 0, cluster_sigma=0.05, outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
    s2 = wl.clustered_scores(4, 48, 3, 0, cluster_sigma=0.05, outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
    np.testing.assert_array_equal(s1, s2)
    assert s1.dtype == np.float32 and not np.array_equal(
        s1, wl.clustered_scores(4, 48, 3, 1, cluster_sigma=0.05, outlier_frac=0.15, outlier_scale=0.3, nu=3.0))


def test_affine_field_and_bf16_bits():
    w = wl.WORKLOADS["tiny"]
    a, b = wl.affine_field(w)
    assert a.shape == (w.elems,) and float(a.max()) <= 0.0 and float(a.min()) >= -1.0
    per = w.elems // w.channels
    assert torch.all(a[:per] == a[0]) and torch.all(b[per:2 * per] == b[per])
    x = torch.randn(4, w.elems)
    torch.testing.assert_close(wl.affine_velocity(x, a, b), a * x + b, rtol=1e-6, atol=1e-7)
    t = torch.tensor([1.0, -2.0, 0.5]).to(torch.bfloat16)
    np.testing.assert_array_equal(wl.bf16_bits(t), np.array([0x3F80, 0xC000, 0x3F00], dtype=np.uint16))


def test_score_distributions_have_the_stated_structure():
    sc = wl.ovf_micro_scores(512, 256)
    assert sc.shape == (512, 256)
    centred = sc - np.median(sc, axis=1, keepdims=True)
    # about 80 % of the scores sit in a narrow cluster (sigma 0.02), the rest are heavy-tailed
    assert 0.7 < np.mean(np.abs(centred) < 0.06) < 0.92
    assert np.abs(centred).max() > 1.0
    w = wl.WORKLOADS["large"]
    assert [w.active_at(s) for s in (0, 1, 2, 4, 5, 7, 8, 27)] == [64, 64, 32, 32, 16, 16, 16, 16]
    assert [w.rows_before(s) for s in (0, 2, 3, 5, 6, 8, 9)] == [64, 64, 32, 32, 16, 16, 16]
