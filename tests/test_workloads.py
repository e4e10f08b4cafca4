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


def test_traffic_ratio_follows_the_committed_profile_and_the_kernel_sources(tmp_path):
    """bench.py takes roofline.traffic from the ncu summary under profiles/ and drops it as soon as
    the kernel sources no longer hash to the value recorded there."""
    import bench
    prof = tmp_path / "step.txt"
    prof.write_text("source_sha256: " + bench._sources_sha256() + "\nalgorithmic_bytes: 1000\n"
                    "  dram__bytes_read.sum    0.600 Kbyte\n  dram__bytes_write.sum   300 byte\n")
    ratio, note = bench.step_traffic_ratio(str(prof))
    assert abs(ratio - 0.9) < 1e-12
    prof.write_text(prof.read_text().replace(bench._sources_sha256(), "0" * 64))
    assert bench.step_traffic_ratio(str(prof))[0] is None
    assert bench.step_traffic_ratio(str(tmp_path / "missing.txt"))[0] is None
    assert isinstance(bench.cpu_model(), str) and bench.cpu_model()


def test_workload_coefficient_sources():
    from dataclasses import replace
    w = wl.WORKLOADS["pro-diffusion"]
    assert w.coef == "ddim" and w.velocity == "eps" and w.vel_dtype == "fp32"
    c = [w.step_coef(s) for s in range(w.n_steps)]
    assert all(cx > 1.0 and cv < 0.0 for cx, cv, _ in c) and c[-1][2] == 0.0 and all(ns > 0 for _, _, ns in c[:-1])
    p_x, p_v = w.preview_coef(30)
    assert p_x > 1.0 and p_v < 0.0
    a, b = wl.eps_mix(w, 30)
    assert abs(a * a + b * b - 1.0) < 1e-12          # (sigma_t, alpha_t) of a variance-preserving schedule
    x = torch.randn(5, w.elems)
    z = wl.normal_noise(wl.scaled(w, n_groups=1), 3, 5)
    v = wl.eps_velocity(x, z, a, b, "fp32")
    torch.testing.assert_close(v, a * x + b * z, rtol=1e-6, atol=1e-7)
    assert wl.eps_velocity(x, z, a, b, "bf16").dtype == torch.bfloat16
    for coef in ("rf-drift", "rf-sde", "vp-em"):
        wc = replace(wl.WORKLOADS["sd15"], coef=coef)
        assert len(wc.step_coef(3)) == 3 and len(wc.preview_coef(3)) == 2
    assert wl.WORKLOADS["large"].step_coef(5) == (1.0, 1.0 / 28, 0.7 * (1.0 / 28) ** 0.5)


def test_config_files_mirror_the_built_in_workloads(tmp_path):
    import glob, json, os
    here = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2512_15347_b200", "configs")
    files = sorted(glob.glob(os.path.join(here, "*.json")))
    names = {os.path.splitext(os.path.basename(f))[0] for f in files}
    assert names == set(wl.WORKLOADS) | {"ovf_micro"}
    for name, w in wl.WORKLOADS.items():
        assert wl.load_workload(os.path.join(here, name + ".json")) == w
    micro = json.load(open(os.path.join(here, "ovf_micro.json")))
    assert {k: micro[k] for k in wl.OVF_MICRO} == wl.OVF_MICRO
    bad = wl.workload_to_dict(wl.WORKLOADS["sd15"])
    bad["stages"] = [[4, 30]]
    p = tmp_path / "bad.json"
    p.write_text(json.dumps(bad))
    import pytest
    with pytest.raises(ValueError):
        wl.load_workload(str(p))
    bad = wl.workload_to_dict(wl.WORKLOADS["sd15"])
    bad["colour"] = "red"
    with pytest.raises(ValueError):
        wl.workload_from_dict(bad)
