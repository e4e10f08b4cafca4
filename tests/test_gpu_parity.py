"""GPU parity: every library call, through the C ABI, against the CPU oracle on the same inputs."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2512_15347_b200 import workloads as wl
from tests import util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2512_15347_b200 import binding
    binding.lib()
    return binding


def _handle(B, G, N0, d, T=4, stages=(), seed=5, bf16=False, **kw):
    cfg = B.make_config(G, N0, d, T, list(stages), seed, B.VEL_BF16 if bf16 else B.VEL_F32, **kw)
    return B.rollout_init(cfg), cfg


# ------------------------------------------------------------------ noise

def test_philox_words_bit_identical(B):
    rng = np.random.default_rng(1)
    n = 1 << 20
    ctr = rng.integers(0, 2**32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
    key = rng.integers(0, 2**32, size=(n, 2), dtype=np.uint64).astype(np.uint32)
    ctr[:3] = [[0, 0, 0, 0], [0xFFFFFFFF] * 4, [0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344]]
    key[:3] = [[0, 0], [0xFFFFFFFF] * 2, [0xA4093822, 0x299F31D0]]
    d_out = torch.empty(n, 4, dtype=torch.int32, device="cuda")
    B.philox_raw(n, U.to_dev(ctr.view(np.int32)), U.to_dev(key.view(np.int32)), d_out)
    got = d_out.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got, oracle.philox_batch(ctr, key))
    assert got[0].tolist() == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]


def test_normals_match_oracle(B):
    seed, step, d = (7 << 32) | 12345, 3, 1 << 16
    ids = np.array([0, 1, 77, 2**31 - 1, 4096], dtype=np.int32)
    out = torch.empty(len(ids), d, device="cuda")
    B.normal_rows(seed, step, 0, len(ids), d, U.to_dev(ids), out)
    got = out.cpu().numpy().astype(np.float64)
    worst = 0.0
    for i, t in enumerate(ids):
        ref = oracle.normal_row(seed, step, int(t), d)
        worst = max(worst, np.abs(got[i] - ref).max())
    # fp32 hardware log2 / sin / cos against fp64: a few ulp of 1 in absolute terms
    assert worst <= 3e-6, worst


# ------------------------------------------------------------------ step

@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("d", [4, 1000, 8192, 3 * 8192 + 20, 65536, 4 * 1024 * 1024 + 8])
def test_step_matches_oracle(B, bf16, d):
    n_groups, n0 = (3, 5) if d < 1 << 20 else (1, 2)      # the 16 MB latents: two rows, 513 chunks each, the last one ragged
    n = n_groups * n0
    rng = np.random.default_rng(d + bf16)
    x = rng.standard_normal((n, d)).astype(np.float32)
    vt = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16 else vt
    v = wl.as_numpy_velocity(vt)
    h, cfg = _handle(B, n_groups, n0, d, seed=99, bf16=bf16)
    try:
        coef = (1.0, 0.05, 0.7 * math.sqrt(0.05))
        x_dev, v_dev = U.to_dev(x), U.vel_to_dev(v)
        x_out = torch.empty_like(x_dev)
        lp = torch.empty(n, device="cuda")
        B.step(h, 0, coef, x_dev, v_dev, None, x_out, lp)
        ref_x, ref_lp = oracle.step(x, v, np.arange(n, dtype=np.int32), 99, 0, *coef)
        assert U.latent_err(x_out.cpu().numpy(), ref_x) <= U.LATENT_TOL
        assert U.logp_err(lp.cpu().numpy(), ref_lp, d) <= U.LOGP_TOL
        # second step in place, general coefficients
        coef2 = (0.98, -0.03, 0.2)
        B.step(h, 1, coef2, x_out, v_dev, None, x_out, lp)
        ref_x2, ref_lp2 = oracle.step(ref_x, v, np.arange(n, dtype=np.int32), 99, 1, *coef2)
        assert U.latent_err(x_out.cpu().numpy(), ref_x2) <= U.LATENT_TOL
        assert U.logp_err(lp.cpu().numpy(), ref_lp2, d) <= U.LOGP_TOL
        # deterministic limit
        B.step(h, 2, (0.5, 0.25, 0.0), x_dev, v_dev, None, x_out, lp)
        ref_x3, ref_lp3 = oracle.step(x, v, np.arange(n, dtype=np.int32), 99, 2, 0.5, 0.25, 0.0)
        assert U.latent_err(x_out.cpu().numpy(), ref_x3) <= 1e-6
        assert np.all(lp.cpu().numpy() == 0.0)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("d", [4, 1000, 3 * 8192 + 20, 262144])
def test_step_with_fused_reward_matches_oracle(B, bf16, d):
    """pg_step_reward: latents and log-probs are pg_step's bit for bit; the reward is the mean of the
    updated latent (the oracle's final-reward stand-in) within the score tolerance; also for the
    deterministic step and with a gather."""
    n_groups, n0 = 3, 4
    n = n_groups * n0
    rng = np.random.default_rng(3 * d + bf16)
    x = rng.standard_normal((n, d)).astype(np.float32) + 0.1
    vt = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16 else vt
    v = wl.as_numpy_velocity(vt)
    x_dev, v_dev = U.to_dev(x), U.vel_to_dev(v)
    for coef in ((1.0, 0.05, 0.15), (1.1, -0.2, 0.3), (0.5, 0.25, 0.0)):
        outs = []
        for fused in (False, True):
            h, _ = _handle(B, n_groups, n0, d, seed=21, bf16=bf16)
            x_out = torch.empty_like(x_dev)
            lp = torch.empty(n, device="cuda")
            rw = torch.full((n,), float("nan"), device="cuda")
            if fused:
                B.step_reward(h, 0, coef, x_dev, v_dev, None, x_out, lp, rw)
            else:
                B.step(h, 0, coef, x_dev, v_dev, None, x_out, lp)
            torch.cuda.synchronize()
            B.rollout_destroy(h)
            outs.append((x_out, lp, rw))
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
        ref_x, ref_lp = oracle.step(x, v, np.arange(n, dtype=np.int32), 21, 0, *coef)
        assert U.latent_err(outs[1][0].cpu().numpy(), ref_x) <= U.LATENT_TOL
        ref_rw = ref_x.astype(np.float64).mean(axis=1)
        assert np.abs(outs[1][2].cpu().numpy() - ref_rw).max() <= U.SCORE_GAP


def test_step_and_score_with_many_short_rows(B):
    """70 000 trajectories of 8 elements: one CTA per row, more rows than a 16-bit grid dimension."""
    G, N0, d = 700, 100, 8
    n = G * N0
    rng = np.random.default_rng(11)
    x = rng.standard_normal((n, d)).astype(np.float32)
    v = rng.standard_normal((n, d)).astype(np.float32)
    h, _ = _handle(B, G, N0, d, seed=4)
    try:
        x_out = torch.empty(n, d, device="cuda")
        lp = torch.empty(n, device="cuda")
        sc = torch.empty(n, device="cuda")
        x_dev, v_dev = U.to_dev(x), U.to_dev(v)
        B.score(h, (1.0, 0.5), x_dev, v_dev, sc)
        B.step(h, 0, (1.0, 0.1, 0.2), x_dev, v_dev, None, x_out, lp)
        ref_x, ref_lp = oracle.step(x, v, np.arange(n, dtype=np.int32), 4, 0, 1.0, 0.1, 0.2)
        assert U.latent_err(x_out.cpu().numpy(), ref_x) <= U.LATENT_TOL
        assert U.logp_err(lp.cpu().numpy(), ref_lp, d) <= U.LOGP_TOL
        assert np.abs(sc.cpu().numpy() - oracle.score(x, v, 1.0, 0.5)[0]).max() <= 1e-6
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_step_is_reproducible_and_mean_mode(B):
    n, d = 6, 5 * 8192
    x = torch.randn(n, d, device="cuda")
    v = torch.randn(n, d, device="cuda")
    outs = []
    for mean_mode in (False, False, True):
        h, _ = _handle(B, 2, 3, d, seed=3, logp_mean=mean_mode)
        x_out = torch.empty_like(x)
        lp = torch.empty(n, device="cuda")
        B.step(h, 0, (1.0, 0.1, 0.3), x, v, None, x_out, lp)
        torch.cuda.synchronize()
        outs.append((x_out.clone(), lp.clone()))
        B.rollout_destroy(h)
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    torch.testing.assert_close(outs[2][1], outs[0][1] / d, rtol=1e-6, atol=0)


# ------------------------------------------------------------------ score

@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("d", [4, 1000, 8192, 3 * 8192 + 20, 262144, 4 * 1024 * 1024 + 8])
def test_score_matches_oracle(B, bf16, d):
    n_groups, n0 = (2, 4) if d < 1 << 20 else (1, 2)
    n = n_groups * n0
    rng = np.random.default_rng(d + 10 * bf16)
    x = rng.standard_normal((n, d)).astype(np.float32) + 0.3
    vt = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16 else vt
    v = wl.as_numpy_velocity(vt)
    h, _ = _handle(B, n_groups, n0, d, bf16=bf16)
    try:
        sc = torch.empty(n, device="cuda")
        prev = torch.empty(n, d, device="cuda")
        x_dev, v_dev = U.to_dev(x), U.vel_to_dev(v)
        B.score(h, (1.0, 0.6), x_dev, v_dev, sc, prev)
        ref, ref_prev = oracle.score(x, v, 1.0, 0.6, want_preview=True)
        assert np.abs(sc.cpu().numpy() - ref).max() <= 1e-6
        assert U.latent_err(prev.cpu().numpy(), ref_prev) <= 1e-6
        sc2 = torch.empty(n, device="cuda")
        B.score(h, (1.0, 0.6), x_dev, v_dev, sc2, None)
        assert torch.equal(sc, sc2)
        B.score(h, (1.0, 0.0), x_dev, None, sc2, None)
        assert np.abs(sc2.cpu().numpy() - x.astype(np.float64).mean(axis=1)).max() <= 1e-6
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


# ------------------------------------------------------------------ OVF

def _ovf_cases():
    rng = np.random.default_rng(42)
    shapes = [(1, 16, 8), (8, 24, 12), (16, 48, 24), (16, 24, 12), (5, 24, 16), (7, 48, 32),
              (7, 32, 8), (3, 64, 8), (64, 64, 32), (64, 32, 16), (64, 16, 16), (9, 256, 32),
              (4, 1, 1), (4, 2, 1), (3, 257, 100), (2, 1024, 1024), (2, 1024, 1), (3, 1000, 500),
              (5, 300, 299)]
    for G, n, k in shapes:
        yield "normal", rng.standard_normal((G, n)).astype(np.float32), k
        yield "ties", rng.integers(0, 4, (G, n)).astype(np.float32), k
        # a few equal scores among distinct ones: a tie sits at one cut of the order in some groups only
        yield "sparse-ties", (np.round(rng.standard_normal((G, n)) * 8) / 8).astype(np.float32), k
        yield "clustered", wl.clustered_scores(G, n, seed=n + k, stage=0, cluster_sigma=0.05,
                                               outlier_frac=0.15, outlier_scale=0.3, nu=3.0), k
    yield "coarse", np.round(rng.standard_normal((512, 32)), 1).astype(np.float32), 16
    yield "equal", np.full((3, 40), 1.25, np.float32), 7
    z = np.zeros((2, 8), np.float32)
    z[:, ::2] = -0.0
    yield "signed-zero", z, 3
    yield "huge", (rng.standard_normal((3, 50)) * 1e37).astype(np.float32), 20
    yield "tiny", (rng.standard_normal((3, 50)) * 1e-40).astype(np.float32), 20


def test_ovf_indices_bit_exact(B):
    for name, sc, k in _ovf_cases():
        G, n = sc.shape
        keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
        kept = torch.empty(G * k, device="cuda")
        adv = torch.empty(G * k, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.ovf_select_batched(G, n, k, U.to_dev(sc), keep, kept, adv, 1e-6, st)
        ref_keep, _ = oracle.ovf_select(sc, k)
        got = keep.cpu().numpy().reshape(G, k)
        np.testing.assert_array_equal(got, ref_keep, err_msg=f"{name} {sc.shape} k={k}")
        ref_kept = np.take_along_axis(sc, ref_keep, axis=1)
        np.testing.assert_array_equal(kept.cpu().numpy().reshape(G, k), ref_kept)
        ref_adv, _, _ = oracle.advantages(ref_kept, 1e-6)
        np.testing.assert_allclose(adv.cpu().numpy().reshape(G, k), ref_adv, rtol=1e-5, atol=1e-6)
        assert int(st.item()) == 0


def test_ovf_non_finite_scores_flagged_and_identical(B):
    sc = np.array([[0.1, np.nan, -np.inf, 0.3, np.inf, 0.2, 0.25, np.nan],
                   [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 8.0]], np.float32)
    for k in range(1, 9):
        keep = torch.empty(2 * k, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.ovf_select_batched(2, 8, k, U.to_dev(sc), keep, None, None, 1e-6, st)
        np.testing.assert_array_equal(keep.cpu().numpy().reshape(2, k), oracle.ovf_select(sc, k)[0])
        assert int(st.item()) == 1


def test_prune_compact_and_ids_through_the_handle(B):
    G, N0, d = 4, 12, 64
    stages = [(1, 7), (2, 7), (3, 3)]
    h, _ = _handle(B, G, N0, d, T=5, stages=stages, seed=1, group_offset=2)
    rng = np.random.default_rng(0)
    try:
        x = torch.randn(G * N0, d, device="cuda")
        v = torch.randn(G * N0, d, device="cuda")
        lp = torch.empty(G * N0, device="cuda")
        B.step(h, 0, (1.0, 0.1, 0.1), x, v, None, x, lp)
        ids_ref = (np.arange(G * N0) + 2 * N0).astype(np.int32)
        rows = x.cpu().numpy()
        k_prev = N0
        for si, (s, k) in enumerate(stages):
            sc = rng.standard_normal((G, k_prev)).astype(np.float32)
            keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
            src = torch.empty(G * k, dtype=torch.int32, device="cuda")
            var = torch.empty(G, device="cuda")
            B.prune_ovf(h, si, U.to_dev(sc), keep, src, var)
            ref_keep, ref_var = oracle.ovf_select(sc, k)
            np.testing.assert_array_equal(keep.cpu().numpy().reshape(G, k), ref_keep)
            np.testing.assert_allclose(var.cpu().numpy(), ref_var, rtol=1e-6, atol=1e-30)
            ref_src = (ref_keep + np.arange(G)[:, None] * k_prev).reshape(-1)
            np.testing.assert_array_equal(src.cpu().numpy(), ref_src)
            # physical compaction of the latent rows and of a narrow per-row array
            cur = U.to_dev(rows)
            dst = torch.empty(G * k, d, device="cuda")
            B.compact(h, keep, cur, dst, d * 4)
            rows = oracle.compact_rows(ref_keep, rows, k_prev)
            np.testing.assert_array_equal(dst.cpu().numpy(), rows)
            narrow = U.to_dev(ids_ref)
            narrow_out = torch.empty(G * k, dtype=torch.int32, device="cuda")
            B.compact(h, keep, narrow, narrow_out, 4)
            ids_ref = oracle.compact_rows(ref_keep, ids_ref.reshape(-1, 1), k_prev).reshape(-1)
            np.testing.assert_array_equal(narrow_out.cpu().numpy(), ids_ref)
            got_ids = torch.empty(G * k, dtype=torch.int32, device="cuda")
            B.rollout_traj_ids(h, got_ids)
            np.testing.assert_array_equal(got_ids.cpu().numpy(), ids_ref)
            # odd row widths take the narrower copy paths
            for width in (6, 100, 40000):
                blob = torch.randint(0, 255, (G * k_prev, width), dtype=torch.uint8, device="cuda")
                blob_out = torch.empty(G * k, width, dtype=torch.uint8, device="cuda")
                B.compact(h, keep, blob, blob_out, width)
                np.testing.assert_array_equal(blob_out.cpu().numpy(),
                                              oracle.compact_rows(ref_keep, blob.cpu().numpy(), k_prev))
            n_act = G * k
            xs = U.to_dev(rows)
            B.step(h, s, (1.0, 0.0, 0.1), xs, xs, None, xs, lp[:n_act])
            rows, _ = oracle.step(rows, rows, ids_ref, 1, s, 1.0, 0.0, 0.1)
            assert U.latent_err(xs.cpu().numpy(), rows) <= U.LATENT_TOL
            k_prev = k
        n_active, next_step, status = B.rollout_status(h)
        assert (n_active, next_step, status) == (G * 3, 4, 0)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_gathered_step_equals_compact_then_step(B):
    G, N0, k, d = 3, 10, 4, 8192 + 256
    h, _ = _handle(B, G, N0, d, T=3, stages=[(0, k)], seed=8, bf16=True)
    try:
        x = torch.randn(G * N0, d, device="cuda")
        v = torch.randn(G * N0, d, device="cuda").to(torch.bfloat16)
        sc = torch.randn(G * N0, device="cuda")
        keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
        src = torch.empty(G * k, dtype=torch.int32, device="cuda")
        B.prune_ovf(h, 0, sc, keep, src, None)
        xg = torch.empty(G * k, d, device="cuda")
        lpg = torch.empty(G * k, device="cuda")
        B.step(h, 0, (1.0, 0.1, 0.2), x, v, src, xg, lpg)
        xc = torch.empty(G * k, d, device="cuda")
        vc = torch.empty(G * k, d, device="cuda", dtype=torch.bfloat16)
        B.compact(h, keep, x, xc, d * 4)
        B.compact(h, keep, v, vc, d * 2)
        ids = torch.empty(G * k, dtype=torch.int32, device="cuda")
        B.rollout_traj_ids(h, ids)
        ref_x, ref_lp = oracle.step(xc.cpu().numpy(), wl.as_numpy_velocity(vc), ids.cpu().numpy(), 8, 0,
                                    1.0, 0.1, 0.2)
        assert U.latent_err(xg.cpu().numpy(), ref_x) <= U.LATENT_TOL
        assert U.logp_err(lpg.cpu().numpy(), ref_lp, d) <= U.LOGP_TOL
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


@pytest.mark.parametrize("G,K", [(1, 8), (8, 12), (16, 12), (4096, 32), (64, 16), (3, 1), (2, 1000)])
def test_advantages_match_oracle(B, G, K):
    rng = np.random.default_rng(G * 1000 + K)
    r = (rng.standard_normal((G, K)) * 0.01 + 0.4).astype(np.float32)
    if G > 2:
        r[1] = 0.5                                   # a constant group: sigma = 0
    h, _ = _handle(B, G, K, 4, adv_eps=1e-6)
    try:
        adv = torch.empty(G * K, device="cuda")
        mean = torch.empty(G, device="cuda")
        std = torch.empty(G, device="cuda")
        B.advantages(h, U.to_dev(r), adv, mean, std)
        ref_adv, ref_mean, ref_std = oracle.advantages(r, 1e-6)
        got = adv.cpu().numpy().reshape(G, K)
        np.testing.assert_allclose(got, ref_adv, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(mean.cpu().numpy(), ref_mean, rtol=1e-6)
        np.testing.assert_allclose(std.cpu().numpy(), ref_std, rtol=1e-6, atol=1e-12)
        assert np.abs(got.mean(axis=1)).max() < 1e-6
        if G > 2:
            assert np.all(got[1] == 0.0)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


# ------------------------------------------------------------------ whole rollouts

@pytest.mark.parametrize("name", ["tiny", "sd15", "pro-diffusion"])
def test_rollout_matches_oracle(B, name):
    w = wl.WORKLOADS[name]
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    ro, out = U.run_gpu(w, inp)
    U.compare_rollouts(w, ref, out)
    if name == "tiny":
        # Config-1 check: the scan's subset attains the exhaustive maximum on the device's scores
        sc = out.stage_scores[0].cpu().numpy()
        best, _ = oracle.ovf_exhaustive(sc, 8)
        kept = sc[out.stage_keep[0].cpu().numpy()]
        assert np.var(kept.astype(np.float64)) == pytest.approx(best, rel=1e-12)
    ro.close()


@pytest.mark.parametrize("name,groups,elems", [("sd3", 4, 16384 + 8192 + 64), ("large", 3, 32768 + 4),
                                               ("pro-standard", 2, 8192 + 64), ("pro-flash", 3, 4096 + 4),
                                               ("pro-diffusion", 2, 2048 + 36)])
def test_scaled_rollout_matches_oracle(B, name, groups, elems):
    w = wl.scaled(wl.WORKLOADS[name], n_groups=groups, elems=elems)
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    ro, out = U.run_gpu(w, inp)
    U.compare_rollouts(w, ref, out)
    n_active, next_step, status = __import__("paper_2512_15347_b200.binding", fromlist=["x"]).rollout_status(ro.h)
    assert (n_active, next_step, status) == (groups * w.final_keep, w.n_steps, 0)
    ro.close()


def test_group_shards_reproduce_the_unsharded_rollout(B):
    """Multi-GPU layout on one device: the groups dealt out to two ranks (3 + 2), each shard run
    with its own handle and global group offset, give the unsharded rollout bit for bit - latents,
    log-probs, kept slots, advantages, trajectory ids."""
    from paper_2512_15347_b200 import sharding
    from paper_2512_15347_b200.rollout import Rollout
    total = 5
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=total, elems=8192 + 512)
    inp = U.SharedInputs(w)
    ro, whole = U.run_gpu(w, inp)
    x0 = U.to_dev(inp.x0)
    parts = []
    for rank in range(2):
        first, count = sharding.group_shard(total, 2, rank)
        sh = Rollout(count, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16,
                     adv_eps=w.adv_eps, group_offset=first)

        def vel(s, x, first=first, count=count):
            per = w.rows_before(s)
            full = U.vel_to_dev(inp.vel_numpy(s, np.empty((total * per, 0))))
            return full[first * per:(first + count) * per].contiguous()

        o = sh.run(x0[first * w.n_expand:(first + count) * w.n_expand], w.step_coef, w.preview_coef, vel)
        torch.cuda.synchronize()
        parts.append((o.x_final.clone(), [t.clone() for t in o.logp], [t.clone() for t in o.stage_keep],
                      o.adv.clone(), o.traj_id.clone()))
        sh.close()
    assert torch.equal(torch.cat([p[0] for p in parts]), whole.x_final)
    for s in range(w.n_steps):
        assert torch.equal(torch.cat([p[1][s] for p in parts]), whole.logp[s])
    for i in range(len(w.stages)):
        assert torch.equal(torch.cat([p[2][i] for p in parts]), whole.stage_keep[i])
    assert torch.equal(torch.cat([p[3] for p in parts]), whole.adv)
    assert torch.equal(torch.cat([p[4] for p in parts]), whole.traj_id)
    ro.close()


def test_resume_from_saved_state(B):
    """Noise is keyed by (seed, trajectory, step, element): restarting from a saved latent at
    step s reproduces the uninterrupted run bit for bit."""
    G, N0, d, T = 2, 6, 4096 + 8, 6
    x0 = torch.randn(G * N0, d, device="cuda")
    v = [torch.randn(G * N0, d, device="cuda") for _ in range(T)]
    lp = torch.empty(G * N0, device="cuda")
    h, _ = _handle(B, G, N0, d, T=T, seed=77)
    x = x0.clone()
    saved = None
    for s in range(T):
        if s == 3:
            saved = x.clone()
        B.step(h, s, (1.0, 0.1, 0.25), x, v[s], None, x, lp)
    torch.cuda.synchronize()
    full, full_lp = x.clone(), lp.clone()
    B.rollout_destroy(h)
    # a fresh handle fast-forwarded with zero-cost steps is not available: the cursor must be
    # walked, so replay steps 0..2 on scratch and continue from the saved latent
    h, _ = _handle(B, G, N0, d, T=T, seed=77)
    scratch = x0.clone()
    for s in range(3):
        B.step(h, s, (1.0, 0.1, 0.25), scratch, v[s], None, scratch, lp)
    x = saved
    for s in range(3, T):
        B.step(h, s, (1.0, 0.1, 0.25), x, v[s], None, x, lp)
    torch.cuda.synchronize()
    assert torch.equal(x, full) and torch.equal(lp, full_lp)
    B.rollout_destroy(h)


def test_host_buffer_rollout_matches_device_rollout(B):
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=2, elems=8192 + 1024)
    inp = U.SharedInputs(w)
    ro, out = U.run_gpu(w, inp)
    cfg = B.make_config(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, B.VEL_BF16,
                        adv_eps=w.adv_eps)
    ws = torch.empty(B.rollout_host_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(inp.x0).pin_memory()
    vels = []
    for s in range(w.n_steps):
        rows = w.n_groups * w.rows_before(s)
        vels.append(U.vel_to_dev(inp.vel_numpy(s, np.empty((rows, 0)))).cpu().pin_memory())
    K = w.final_keep
    x_final = torch.empty(w.n_groups * K, w.elems).pin_memory()
    logp = torch.empty(w.traj_steps).pin_memory()
    keep = torch.empty(sum(w.n_groups * k for _, k in w.stages), dtype=torch.int32).pin_memory()
    adv = torch.empty(w.n_groups * K).pin_memory()
    ids = torch.empty(w.n_groups * K, dtype=torch.int32).pin_memory()
    rc = B.rollout_host(cfg, [w.step_coef(s) for s in range(w.n_steps)],
                        [w.preview_coef(s) for s, _ in w.stages], x0, vels, None, None,
                        x_final, logp, keep, adv, ids, ws)
    assert rc == 0
    assert torch.equal(x_final, out.x_final.cpu())
    assert torch.equal(logp, torch.cat(out.logp).cpu())
    assert torch.equal(keep, torch.cat(out.stage_keep).cpu())
    assert torch.equal(adv, out.adv.cpu())
    assert torch.equal(ids, out.traj_id.cpu())
    # the same on an existing handle, twice in a row (the second call reuses the handle's streams
    # and events and finds the cursor at the end of the first rollout)
    h = B.rollout_init(cfg)
    args = B.HostArgs([w.step_coef(s) for s in range(w.n_steps)], [w.preview_coef(s) for s, _ in w.stages], vels)
    for _ in range(2):
        for t in (x_final, logp, adv):
            t.fill_(float("nan"))
        keep.fill_(-1)
        ids.fill_(-1)
        assert B.rollout_host_on(h, args, x0, None, x_final, logp, keep, adv, ids, ws) == 0
        assert torch.equal(x_final, out.x_final.cpu()) and torch.equal(logp, torch.cat(out.logp).cpu())
        assert torch.equal(keep, torch.cat(out.stage_keep).cpu()) and torch.equal(adv, out.adv.cpu())
        assert torch.equal(ids, out.traj_id.cpu())
    assert B.rollout_status(h) == (w.n_groups * K, w.n_steps, 0)
    B.rollout_destroy(h)
    ro.close()


def test_host_buffer_rollout_draws_its_own_initial_latents(B):
    """x0 = NULL: the library draws x_0 ~ N(0, I) on the device (noise stream 1).  The result is
    the rollout that starts from those rows handed in as a host buffer, bit for bit, and the rows
    themselves are the oracle's normals for that stream."""
    from paper_2512_15347_b200.rollout import initial_latents
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=2, elems=8192 + 1024)
    inp = U.SharedInputs(w)
    offset = 3
    cfg = B.make_config(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, B.VEL_BF16,
                        adv_eps=w.adv_eps, group_offset=offset)
    ws = torch.empty(B.rollout_host_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    x0_dev = initial_latents(w.seed, w.n_groups, w.n_expand, w.elems, group_offset=offset)
    for row in (0, w.n_groups * w.n_expand - 1):
        ref = oracle.normal_row(w.seed, 0, offset * w.n_expand + row, w.elems, stream=1)
        assert np.abs(x0_dev[row].cpu().numpy() - ref).max() <= 3e-6
    vels = []
    for s in range(w.n_steps):
        rows = w.n_groups * w.rows_before(s)
        vels.append(U.vel_to_dev(inp.vel_numpy(s, np.empty((rows, 0)))).cpu().pin_memory())
    K = w.final_keep
    coefs = [w.step_coef(s) for s in range(w.n_steps)]
    pcoefs = [w.preview_coef(s) for s, _ in w.stages]

    def run(x0):
        res = (torch.empty(w.n_groups * K, w.elems).pin_memory(), torch.empty(w.traj_steps).pin_memory(),
               torch.empty(sum(w.n_groups * k for _, k in w.stages), dtype=torch.int32).pin_memory(),
               torch.empty(w.n_groups * K).pin_memory(),
               torch.empty(w.n_groups * K, dtype=torch.int32).pin_memory())
        assert B.rollout_host(cfg, coefs, pcoefs, x0, vels, None, None, *res, ws) == 0
        return res

    drawn = run(None)
    given = run(x0_dev.cpu().pin_memory())
    for a, b in zip(drawn, given):
        assert torch.equal(a, b)
    assert torch.isfinite(drawn[0]).all() and drawn[4].min() >= offset * w.n_expand


# ------------------------------------------------------------------ call-order and argument errors

def test_out_of_sequence_calls_are_refused(B):
    G, N0, d = 2, 8, 64
    h, _ = _handle(B, G, N0, d, T=4, stages=[(1, 4)])
    x = torch.zeros(G * N0, d, device="cuda")
    lp = torch.empty(G * N0, device="cuda")
    keep = torch.empty(G * 4, dtype=torch.int32, device="cuda")
    sc = torch.zeros(G * N0, device="cuda")
    try:
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, 0.1), x, x, None, x, lp)           # step 0 not taken yet
        assert e.value.code == B.ESTATE
        with pytest.raises(B.PgError) as e:
            B.prune_ovf(h, 0, sc, keep)                            # stage 0 belongs to step 1
        assert e.value.code == B.ESTATE
        with pytest.raises(B.PgError) as e:
            B.compact(h, keep, x, x.clone(), d * 4)                 # nothing pruned yet
        assert e.value.code == B.ESTATE
        B.step(h, 0, (1, 0, 0.1), x, x, None, x, lp)
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, 0.1), x, x, None, x, lp)           # must prune before step 1
        assert e.value.code == B.ESTATE
        with pytest.raises(B.PgError) as e:
            B.prune_ovf(h, 1, sc, keep)                            # no such stage
        assert e.value.code == B.ESTATE
        src = torch.empty(G * 4, dtype=torch.int32, device="cuda")
        B.prune_ovf(h, 0, sc, keep, src)
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, 0.1), x, x, src, x, lp)            # gather must not be in place
        assert e.value.code == B.EINVAL
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, 0.1), x, x, src, x[2:], lp)        # nor into an offset view of its input
        assert e.value.code == B.EINVAL
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, -0.1), x, x, None, x, lp)          # negative noise scale
        assert e.value.code == B.EINVAL
        with pytest.raises(B.PgError) as e:
            B.step(h, 1, (1, 0, 0.1), x[0, 1:], x, None, x, lp)    # misaligned pointer
        assert e.value.code == B.EINVAL
        with pytest.raises(B.PgError) as e:
            B.compact(h, keep, x, x[1:], d * 4)                     # overlapping source / destination
        assert e.value.code == B.EINVAL
        y = torch.empty(G * 4, d, device="cuda")
        B.step(h, 1, (1, 0, 0.1), x, x, src, y, lp)
        assert B.rollout_status(h) == (G * 4, 2, 0)
        # the device is still healthy after all refusals
        B.rollout_reset(h)
        assert B.rollout_status(h) == (G * N0, 0, 0)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


@pytest.mark.parametrize("name,coef,eta,groups,elems", [
    ("pro-diffusion", "ddim", 0.5, 3, 16384),          # DDIM with partial stochasticity, full-length SD latents
    ("pro-diffusion", "vp-em", 1.0, 2, 8192 + 36),     # Euler-Maruyama of the VP reverse SDE
    ("pro-standard", "rf-sde", 1.0, 2, 32768 + 4),     # rectified flow with the score-corrected drift
    ("large", "ddim", 1.0, 2, 65536 + 8),              # early checkpoints: large preview coefficients
])
def test_rollout_under_other_backbones_matches_oracle(B, name, coef, eta, groups, elems):
    """Coefficients of the diffusion branch (Eq. dm_sde, epsilon prediction: c_x != 1, c_v < 0, a
    noise level that changes from step to step, clean-sample or probability-flow previews) and of
    the score-corrected rectified flow cross the C ABI and give the oracle's rollout."""
    from dataclasses import replace
    w = replace(wl.scaled(wl.WORKLOADS[name], n_groups=groups, elems=elems), coef=coef, eta=eta)
    if coef != "rf-sde":
        w = replace(w, velocity="eps", vel_dtype="fp32")     # stand-in noise-prediction network in the loop
    c = [w.step_coef(s) for s in range(w.n_steps)]
    assert all(abs(cx - 1.0) > 1e-3 for cx, _, _ in c)              # never the unit-c_x fast path
    if coef != "rf-sde":
        assert all(cv < 0 for _, cv, _ in c) and len({ns for _, _, ns in c}) == w.n_steps
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    ro, out = U.run_gpu(w, inp)
    U.compare_rollouts(w, ref, out)
    assert B.rollout_status(ro.h) == (groups * w.final_keep, w.n_steps, 0)
    ro.close()


# ------------------------------------------------------------------ edge schedules

@pytest.mark.parametrize("groups,n0,stages,T,d,vdt", [
    (2, 6, (), 3, 4, "fp32"),                         # no pruning at all, shortest latent
    (3, 7, ((0, 3),), 4, 12, "bf16"),                 # pruning before the very first step
    (2, 9, ((1, 9), (2, 1)), 4, 8192 + 4, "fp32"),    # identity stage, then a single survivor
    (1, 1, ((0, 1),), 2, 8, "fp32"),                  # one trajectory
    (2, 1024, ((1, 1024), (2, 300), (3, 256)), 5, 4, "fp32"),   # largest group: CTA and warp selection
    (5, 33, ((2, 32), (3, 2)), 5, 260, "bf16"),       # sizes straddling the lane-count boundaries
])
def test_edge_schedules_match_oracle(B, groups, n0, stages, T, d, vdt):
    w = wl.Workload("edge", groups, n0, tuple(stages), T, d, 1, vdt, 11, "normal", "preview")
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    ro, out = U.run_gpu(w, inp)
    U.compare_rollouts(w, ref, out)
    assert B.rollout_status(ro.h) == (groups * w.final_keep, T, 0)
    ro.close()


def test_empty_batches_are_accepted(B):
    keep = torch.empty(0, dtype=torch.int32, device="cuda")
    sc = torch.empty(0, device="cuda")
    B.ovf_select_batched(0, 8, 4, sc, keep)
    B.philox_raw(0, None, None, None)
    B.normal_rows(1, 0, 0, 0, 8, None, None)
    B.score_static(0, 8, B.VEL_F32, (1.0, 0.0), None, None, None)
    torch.cuda.synchronize()


def test_survivor_rows_match_oracle_on_random_schedules(B):
    rng = np.random.default_rng(5)
    for trial in range(12):
        G = int(rng.integers(1, 6))
        N0 = int(rng.integers(1, 40))
        T = int(rng.integers(1, 12))
        n_st = int(rng.integers(0, min(T, 4) + 1))
        steps = sorted(rng.choice(T, size=n_st, replace=False).tolist())
        stages, keeps, k_prev = [], [], N0
        for s_ in steps:
            k = int(rng.integers(1, k_prev + 1))
            stages.append((int(s_), k))
            keeps.append(np.stack([np.sort(rng.choice(k_prev, size=k, replace=False)) for _ in range(G)]).astype(np.int32))
            k_prev = k
        h, _ = _handle(B, G, N0, 8, T=T, stages=stages)
        try:
            packed = np.concatenate([k.reshape(-1) for k in keeps]) if keeps else np.zeros(1, np.int32)
            rows = torch.full((T, G * k_prev), -1, dtype=torch.int32, device="cuda")
            B.survivor_rows(h, U.to_dev(packed) if keeps else None, rows)
            ref = oracle.survivor_rows(G, N0, T, stages, keeps)
            np.testing.assert_array_equal(rows.cpu().numpy(), ref, err_msg=f"trial {trial}: {stages}")
            assert B.rollout_status(h)[2] == 0
        finally:
            torch.cuda.synchronize()
            B.rollout_destroy(h)


def test_survivors_history_after_a_pruned_rollout(B):
    """After a rollout with three prunes: the survivors' log-prob history and their latents of an
    early step, collected through pg_survivor_rows / _logp / pg_gather_rows, against the oracle's."""
    from paper_2512_15347_b200.rollout import NativeRollout
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=3, elems=8192 + 256)
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp, keep_steps=True)
    ro, out = U.run_gpu(w, inp)
    T, n_final = w.n_steps, w.n_groups * w.final_keep
    keep_packed = torch.cat(out.stage_keep)
    logp_packed = torch.cat(out.logp)
    rows = torch.empty(T, n_final, dtype=torch.int32, device="cuda")
    hist = torch.empty(T, n_final, device="cuda")
    B.survivor_rows(ro.h, keep_packed, rows)
    B.survivor_logp(ro.h, rows, logp_packed, hist)
    own_keep = [a.cpu().numpy().reshape(w.n_groups, -1) for a in out.stage_keep]
    np.testing.assert_array_equal(rows.cpu().numpy(),
                                  oracle.survivor_rows(w.n_groups, w.n_expand, T, w.stages, own_keep))
    # the values below need the device's selections to be the oracle's (they are, bit-reproducibly,
    # for this seed; a score gap below the score tolerance could legitimately flip one)
    assert all(np.array_equal(a, b) for a, b in zip(own_keep, ref.stage_keep))
    ref_rows = oracle.survivor_rows(w.n_groups, w.n_expand, T, w.stages, ref.stage_keep)
    ref_hist = np.stack([ref.logp[t][ref_rows[t]] for t in range(T)])
    assert U.logp_err(hist.cpu().numpy(), ref_hist, w.elems) <= U.LOGP_TOL
    # the survivors' latents entering step 1 (stored in the 64-per-group layout of step 0)
    x1 = torch.empty(w.n_groups * w.n_expand, w.elems, device="cuda")
    lp = torch.empty(w.n_groups * w.n_expand, device="cuda")
    B.rollout_reset(ro.h)
    B.step(ro.h, 0, w.step_coef(0), U.to_dev(inp.x0), inp.vel_device(0, torch.empty(w.n_groups * w.n_expand, 0)),
           None, x1, lp)
    surv = torch.empty(n_final, w.elems, device="cuda")
    B.gather_rows(ro.h, rows[0], n_final, w.n_groups * w.n_expand, x1, surv, w.elems * 4)
    assert U.latent_err(surv.cpu().numpy(), ref.x_steps[0][ref_rows[0]]) <= U.LATENT_TOL
    assert B.rollout_status(ro.h)[2] == 0
    # an index outside the source is skipped and reported
    bad = rows[0].clone()
    bad[3] = w.n_groups * w.n_expand
    surv.fill_(7.0)
    B.gather_rows(ro.h, bad, n_final, w.n_groups * w.n_expand, x1, surv, w.elems * 4)
    with pytest.raises(B.PgError) as e:
        B.rollout_status(ro.h)
    assert e.value.code == B.EINDEX
    assert torch.all(surv[3] == 7.0)
    ro.close()


def test_bounded_wait_runs_out_and_is_reported(B):
    """The device-side wait gives up instead of hanging: a wait that nothing completes ends by
    itself, the status word reports it, and the handle stays usable afterwards."""
    G, N0, d = 2, 8, 64
    h, _ = _handle(B, G, N0, d, T=2, stages=[(0, 4)])
    try:
        assert B.rollout_status(h) == (G * N0, 0, 0)
        B.selftest_bounded_wait(h)
        with pytest.raises(B.PgError) as e:
            B.rollout_status(h)
        assert e.value.code == B.ETIMEOUT
        assert B.rollout_status(h, raise_on_flags=False)[2] == 2
        B.rollout_reset(h)
        sc = np.arange(G * N0, dtype=np.float32).reshape(G, N0)
        keep = torch.empty(G * 4, dtype=torch.int32, device="cuda")
        B.prune_ovf(h, 0, U.to_dev(sc), keep)
        assert B.rollout_status(h) == (G * 4, 0, 0)
        np.testing.assert_array_equal(keep.cpu().numpy().reshape(G, 4), oracle.ovf_select(sc, 4)[0])
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


# ------------------------------------------------------------------ diagnostics and the uniform baseline

def test_group_stats_match_oracle(B):
    for G, n in [(1, 16), (64, 64), (4096, 256), (7, 1000), (3, 1)]:
        sc = wl.clustered_scores(G, n, G + n, 0, cluster_sigma=0.05, outlier_frac=0.15,
                                 outlier_scale=0.3, nu=3.0)
        mean = torch.empty(G, device="cuda")
        std = torch.empty(G, device="cuda")
        frac = torch.empty(G, device="cuda")
        for delta in (0.5, 1.0):
            B.group_stats(G, n, U.to_dev(sc), delta, mean, std, frac)
            rm, rs, rf = oracle.group_stats(sc, delta)
            np.testing.assert_allclose(mean.cpu().numpy(), rm, rtol=1e-6, atol=1e-7)
            np.testing.assert_allclose(std.cpu().numpy(), rs, rtol=1e-6, atol=1e-12)
            np.testing.assert_allclose(frac.cpu().numpy(), rf, rtol=1e-6, atol=1e-7)


def test_uniform_pruning_matches_oracle_bit_for_bit(B):
    G, N0, d = 5, 48, 16
    stages = [(0, 32), (1, 8), (2, 8)]
    h, _ = _handle(B, G, N0, d, T=4, stages=stages, seed=(9 << 32) | 77, group_offset=3)
    try:
        x = torch.randn(G * N0, d, device="cuda")
        lp = torch.empty(G * N0, device="cuda")
        ids_ref = (np.arange(G * N0) + 3 * N0).astype(np.int32)
        k_prev = N0
        for si, (s, k) in enumerate(stages):
            keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
            src = torch.empty(G * k, dtype=torch.int32, device="cuda")
            B.prune_uniform(h, si, keep, src)
            ref_keep = oracle.select_uniform(G, k_prev, k, (9 << 32) | 77, si, group_offset=3)
            np.testing.assert_array_equal(keep.cpu().numpy().reshape(G, k), ref_keep)
            np.testing.assert_array_equal(src.cpu().numpy(),
                                          (ref_keep + np.arange(G)[:, None] * k_prev).reshape(-1))
            ids_ref = oracle.compact_rows(ref_keep, ids_ref.reshape(-1, 1), k_prev).reshape(-1)
            got_ids = torch.empty(G * k, dtype=torch.int32, device="cuda")
            B.rollout_traj_ids(h, got_ids)
            np.testing.assert_array_equal(got_ids.cpu().numpy(), ids_ref)
            y = torch.empty(G * k, d, device="cuda")
            B.step(h, s, (1.0, 0.0, 0.1), x, x, src, y, lp[: G * k])
            x = y
            k_prev = k
        assert B.rollout_status(h) == (G * 8, 3, 0)
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_host_buffer_rollout_with_external_scores_and_rewards(B):
    """pg_rollout_host fed with reward-model style inputs: per-stage scores and final rewards from
    the host instead of the preview mean."""
    w = wl.scaled(wl.WORKLOADS["sd3"], n_groups=3, elems=4096 + 64)
    inp = U.SharedInputs(w)
    ref = U.run_oracle(w, inp)
    cfg = B.make_config(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, B.VEL_BF16,
                        adv_eps=w.adv_eps)
    ws = torch.empty(B.rollout_host_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    x0 = torch.from_numpy(inp.x0).pin_memory()
    vels = [U.vel_to_dev(inp.vel_numpy(s, np.empty((w.n_groups * w.rows_before(s), 0)))).cpu().pin_memory()
            for s in range(w.n_steps)]
    # the stand-in reward model is keyed by original trajectory: replay the oracle's survivors
    stage_ids = [np.arange(w.n_groups * w.n_expand, dtype=np.int32)]
    for keep, (s, k) in zip(ref.stage_keep, w.stages):
        prev = stage_ids[-1].reshape(w.n_groups, -1)
        stage_ids.append(np.take_along_axis(prev, keep, axis=1).reshape(-1))
    stage_scores = [torch.from_numpy(wl.sd3_stage_scores(w, i, stage_ids[i])).pin_memory()
                    for i in range(len(w.stages))]
    final = torch.from_numpy(wl.sd3_stage_scores(w, 99, stage_ids[-1])).pin_memory()
    K = w.final_keep
    x_final = torch.empty(w.n_groups * K, w.elems).pin_memory()
    logp = torch.empty(w.traj_steps).pin_memory()
    keep = torch.empty(sum(w.n_groups * k for _, k in w.stages), dtype=torch.int32).pin_memory()
    adv = torch.empty(w.n_groups * K).pin_memory()
    ids = torch.empty(w.n_groups * K, dtype=torch.int32).pin_memory()
    rc = B.rollout_host(cfg, [w.step_coef(s) for s in range(w.n_steps)], [], x0, vels, stage_scores,
                        final, x_final, logp, keep, adv, ids, ws)
    assert rc == 0
    np.testing.assert_array_equal(keep.numpy(), np.concatenate([k.reshape(-1) for k in ref.stage_keep]))
    np.testing.assert_array_equal(ids.numpy(), ref.traj_id)
    assert U.latent_err(x_final.numpy(), ref.x_final) <= U.LATENT_TOL
    assert U.logp_err(logp.numpy(), np.concatenate(ref.logp), w.elems) <= U.LOGP_TOL
    np.testing.assert_allclose(adv.numpy().reshape(w.n_groups, K), ref.adv, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("bf16_vel", [False, True])
@pytest.mark.parametrize("d", [4, 3 * 8192 + 20])
def test_preview_emission_matches_oracle(B, bf16_vel, d):
    n_groups, n0 = 2, 5
    n = n_groups * n0
    rng = np.random.default_rng(d)
    x = rng.standard_normal((n, d)).astype(np.float32)
    vt = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16_vel else vt
    v = wl.as_numpy_velocity(vt)
    h, _ = _handle(B, n_groups, n0, d, bf16=bf16_vel)
    try:
        _, ref = oracle.score(x, v, 0.9, 0.4, want_preview=True)
        out32 = torch.empty(n, d, device="cuda")
        out16 = torch.empty(n, d, device="cuda", dtype=torch.bfloat16)
        B.preview(h, (0.9, 0.4), U.to_dev(x), U.vel_to_dev(v), out32)
        B.preview(h, (0.9, 0.4), U.to_dev(x), U.vel_to_dev(v), out16)
        assert U.latent_err(out32.cpu().numpy(), ref) <= 1e-6
        # bf16: 8 significant bits, round to nearest
        assert U.latent_err(out16.float().cpu().numpy(), ref) <= 2.0 ** -8
        assert torch.equal(out16, out32.to(torch.bfloat16))
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


@pytest.mark.parametrize("bf16_vel", [False, True])
@pytest.mark.parametrize("d", [4, 1000, 3 * 8192 + 20, 262144])
def test_score_with_bf16_preview_in_one_pass_matches_oracle(B, bf16_vel, d):
    """pg_score_preview: the scores are pg_score's bit for bit and the oracle's within the score
    tolerance; the bf16 preview is the fp32 preview rounded to nearest even, i.e. the oracle's
    preview to 8 significant bits."""
    n_groups, n0 = 3, 4
    n = n_groups * n0
    rng = np.random.default_rng(d + 7 * bf16_vel)
    x = rng.standard_normal((n, d)).astype(np.float32) - 0.2
    vt = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16_vel else vt
    v = wl.as_numpy_velocity(vt)
    h, _ = _handle(B, n_groups, n0, d, bf16=bf16_vel)
    try:
        coef = (2.27, -2.04)          # a clean-sample preview of the diffusion branch
        ref, ref_prev = oracle.score(x, v, *coef, want_preview=True)
        x_dev, v_dev = U.to_dev(x), U.vel_to_dev(v)
        sc16, sc32, sc0 = (torch.empty(n, device="cuda") for _ in range(3))
        out16 = torch.full((n, d), float("nan"), device="cuda", dtype=torch.bfloat16)
        out32 = torch.empty(n, d, device="cuda")
        B.score_preview(h, coef, x_dev, v_dev, sc16, out16)
        B.score_preview(h, coef, x_dev, v_dev, sc32, out32)
        B.score(h, coef, x_dev, v_dev, sc0)
        assert torch.equal(sc16, sc0) and torch.equal(sc32, sc0)
        # the preview has rms ~3: the score tolerance scales with it
        assert np.abs(sc16.cpu().numpy() - ref).max() <= 3e-6
        assert U.latent_err(out32.cpu().numpy(), ref_prev) <= 1e-6
        assert torch.equal(out16, out32.to(torch.bfloat16))
        assert U.latent_err(out16.float().cpu().numpy(), ref_prev) <= 2.0 ** -8
        # without a velocity term
        B.score_preview(h, (0.5, 0.0), x_dev, None, sc16, out16)
        assert torch.equal(out16, (0.5 * x_dev).to(torch.bfloat16))
        assert np.abs(sc16.cpu().numpy() - 0.5 * x.astype(np.float64).mean(axis=1)).max() <= 1e-6
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_ovf_misaligned_and_ragged_score_rows(B):
    """Score rows that cannot be staged with a bulk copy (base not 16-byte aligned, or a CTA's rows
    not a multiple of 16 bytes) take the ordinary-load path and give the same selection."""
    rng = np.random.default_rng(5)
    for G, n, k in [(9, 25, 7), (6, 256, 32), (5, 3, 2), (4, 64, 16), (7, 31, 31)]:
        sc = rng.standard_normal((G, n)).astype(np.float32)
        ref_keep, _ = oracle.ovf_select(sc, k)
        for shift in (0, 1, 2):
            buf = torch.zeros(G * n + 4, device="cuda")
            view = buf[shift: shift + G * n]
            view.copy_(torch.from_numpy(sc).reshape(-1))
            keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
            B.ovf_select_batched(G, n, k, view, keep)
            np.testing.assert_array_equal(keep.cpu().numpy().reshape(G, k), ref_keep)


def test_native_rollout_and_graph_replay_equal_the_stepwise_driver(B):
    from paper_2512_15347_b200.rollout import NativeRollout
    w = wl.scaled(wl.WORKLOADS["large"], n_groups=3, elems=8192 + 256)
    inp = U.SharedInputs(w)
    ro, out = U.run_gpu(w, inp)
    want = (out.x_final.clone(), torch.cat(out.logp).clone(), torch.cat(out.stage_keep).clone(),
            out.adv.clone(), out.traj_id.clone())
    vels = [U.vel_to_dev(inp.vel_numpy(s, np.empty((w.n_groups * w.rows_before(s), 0))))
            for s in range(w.n_steps)]
    nat = NativeRollout(ro, [w.step_coef(s) for s in range(w.n_steps)],
                        [w.preview_coef(s) for s, _ in w.stages], vels)
    x0 = U.to_dev(inp.x0)

    def check(o):
        torch.cuda.synchronize()
        assert torch.equal(o.x_final, want[0])
        assert torch.equal(torch.cat(o.logp), want[1])
        assert torch.equal(torch.cat(o.stage_keep), want[2])
        assert torch.equal(o.adv, want[3])
        assert torch.equal(o.traj_id, want[4])

    check(nat.run(x0))
    nat.capture(x0)
    for _ in range(3):
        nat.ws.zero_()                      # results must be rebuilt by the replay alone
        check(nat.replay())
    assert B.rollout_status(ro.h) == (w.n_groups * w.final_keep, w.n_steps, 0)
    ro.close()


def test_out_of_range_gather_indices_are_reported_not_dereferenced(B):
    G, N0, k, d = 2, 8, 4, 8192 + 64
    h, _ = _handle(B, G, N0, d, T=3, stages=[(0, k)], seed=4)
    try:
        x = torch.randn(G * N0, d, device="cuda")
        sc = torch.randn(G * N0, device="cuda")
        keep = torch.empty(G * k, dtype=torch.int32, device="cuda")
        src = torch.empty(G * k, dtype=torch.int32, device="cuda")
        B.prune_ovf(h, 0, sc, keep, src)
        good_src = src.clone()
        bad = src.clone()
        bad[1] = 10 ** 6
        bad[5] = -1
        y_bad = torch.zeros(G * k, d, device="cuda")
        y_good = torch.zeros(G * k, d, device="cuda")
        lp = torch.empty(G * k, device="cuda")
        B.step(h, 0, (1.0, 0.1, 0.2), x, x, bad, y_bad, lp)
        n_active, next_step, status = B.rollout_status(h, raise_on_flags=False)
        assert status & 4 and next_step == 1
        with pytest.raises(B.PgError) as e:
            B.rollout_status(h)
        assert e.value.code == B.EINDEX
        # the rows with valid indices are unaffected (same noise: same trajectory ids and step)
        B.rollout_reset(h)
        B.prune_ovf(h, 0, sc, keep, src)
        B.step(h, 0, (1.0, 0.1, 0.2), x, x, good_src, y_good, lp)
        ok_rows = [i for i in range(G * k) if i not in (1, 5)]
        assert torch.equal(y_bad[ok_rows], y_good[ok_rows])
        assert B.rollout_status(h)[2] == 0
        # compaction: a bad slot is skipped and reported
        bad_keep = keep.clone()
        bad_keep[2] = N0 + 3
        dst = torch.full((G * k, d), -7.0, device="cuda")
        B.compact(h, bad_keep, x, dst, d * 4)
        assert B.rollout_status(h, raise_on_flags=False)[2] & 4
        assert torch.all(dst[2] == -7.0) and torch.equal(dst[0], x[int(keep[0])])
        narrow = torch.full((G * k,), -1, dtype=torch.int32, device="cuda")
        B.compact(h, bad_keep, torch.arange(G * N0, dtype=torch.int32, device="cuda"), narrow, 4)
        torch.cuda.synchronize()
        assert int(narrow[2]) == -1 and int(narrow[0]) == int(keep[0])
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_graphed_stepwise_rollout_with_a_network_in_the_loop(B):
    """The tiny workload (predictions computed from the current latents by torch ops) captured
    into a CUDA graph: replays reproduce the step-by-step run bit for bit, also after x0 changes."""
    from paper_2512_15347_b200.rollout import GraphedRollout
    w = wl.WORKLOADS["tiny"]
    inp = U.SharedInputs(w)
    ro, out = U.run_gpu(w, inp)
    want = [t.clone() for t in (out.x_final, torch.cat(out.logp), out.stage_keep[0], out.adv, out.traj_id)]
    a, b = (t.cuda() for t in inp.affine)
    x0 = U.to_dev(inp.x0)
    g = GraphedRollout(ro, x0, w.step_coef, w.preview_coef, lambda s, x: wl.affine_velocity(x, a, b))

    def same(o, ref):
        torch.cuda.synchronize()
        got = (o.x_final, torch.cat(o.logp), o.stage_keep[0], o.adv, o.traj_id)
        return all(torch.equal(p, q) for p, q in zip(got, ref))

    assert same(g.replay(), want) and same(g.replay(), want)
    x0.mul_(-1.0)                                      # new initial latents, same graph
    o = g.replay()
    torch.cuda.synchronize()
    assert not torch.equal(o.x_final, want[0])
    ro2, out2 = U.run_gpu(w, type("I", (), {"x0": -inp.x0, "vel_device": inp.vel_device})())
    assert same(o, (out2.x_final, torch.cat(out2.logp), out2.stage_keep[0], out2.adv, out2.traj_id))
    ro2.close()
    ro.close()


def test_initial_latents_from_the_library_generator(B):
    from paper_2512_15347_b200.rollout import initial_latents
    G, N0, d = 3, 5, 4096
    x = initial_latents(17, G, N0, d, group_offset=2).cpu().numpy()
    for row in (0, 7, 14):
        ref = oracle.normal_row(17, 0, 2 * N0 + row, d, stream=1)
        assert np.abs(x[row] - ref).max() <= 3e-6
    # a shard draws the rows of the whole batch
    whole = initial_latents(17, 5, N0, d).cpu().numpy()
    np.testing.assert_array_equal(x, whole[2 * N0:])
    # stream 1 differs from the SDE noise stream of step 0
    assert np.abs(x[0] - oracle.normal_row(17, 0, 2 * N0, d, stream=0)).max() > 1.0
    assert abs(x.mean()) < 0.02 and abs(x.std() - 1.0) < 0.02
    # many rows (more than one grid dimension used to allow)
    ids = torch.arange(70000, dtype=torch.int32, device="cuda")
    out = torch.empty(70000, 4, device="cuda")
    B.normal_rows(1, 0, 1, 70000, 4, ids, out)
    np.testing.assert_allclose(out[69999].cpu().numpy(), oracle.normal_row(1, 0, 69999, 4, stream=1), atol=3e-6)


def test_checkpoint_restore_continues_bit_for_bit(B):
    """Save (latents, cursor, trajectory ids) after a prune, restore them into a fresh handle and
    finish the schedule: identical to the uninterrupted run."""
    G, N0, d, T = 3, 10, 8192 + 128, 6
    stages = [(1, 6), (4, 2)]
    x0 = torch.randn(G * N0, d, device="cuda")
    vels = [torch.randn(G * N0, d, device="cuda") for _ in range(T)]
    scores = [torch.randn(G * N0, device="cuda") for _ in stages]

    def run(h, x, start, stages_done, stop):
        lp = torch.empty(G * N0, device="cuda")
        k = N0 if stages_done == 0 else stages[stages_done - 1][1]
        si = stages_done
        for s in range(start, stop):
            src = None
            if si < len(stages) and stages[si][0] == s:
                k_new = stages[si][1]
                keep = torch.empty(G * k_new, dtype=torch.int32, device="cuda")
                src = torch.empty(G * k_new, dtype=torch.int32, device="cuda")
                B.prune_ovf(h, si, scores[si][: G * k], keep, src)
                k, si = k_new, si + 1
            y = torch.empty(G * k, d, device="cuda")
            B.step(h, s, (1.0, 0.1, 0.3), x, vels[s], src, y, lp[: G * k])
            x = y
        return x, lp[: G * k].clone(), si

    h, _ = _handle(B, G, N0, d, T=T, stages=stages, seed=31)
    full_x, full_lp, _ = run(h, x0, 0, 0, T)
    torch.cuda.synchronize()
    B.rollout_destroy(h)

    h, _ = _handle(B, G, N0, d, T=T, stages=stages, seed=31)
    mid_x, _, done = run(h, x0, 0, 0, 3)                  # stops after step 2 (first prune done)
    ids = torch.empty(G * 6, dtype=torch.int32, device="cuda")
    B.rollout_traj_ids(h, ids)
    saved = (mid_x.clone(), ids.clone(), 3, done)
    torch.cuda.synchronize()
    B.rollout_destroy(h)

    h, _ = _handle(B, G, N0, d, T=T, stages=stages, seed=31)
    with pytest.raises(B.PgError) as e:
        B.rollout_restore(h, 3, 0, saved[1])                # stage at step 1 cannot be pending at step 3
    assert e.value.code == B.ESTATE
    B.rollout_restore(h, saved[2], saved[3], saved[1])
    assert B.rollout_status(h) == (G * 6, 3, 0)
    x, lp, _ = run(h, saved[0], 3, saved[3], T)
    torch.cuda.synchronize()
    assert torch.equal(x, full_x) and torch.equal(lp, full_lp)
    B.rollout_destroy(h)


def test_ovf_survivors_are_more_spread_out_than_uniform_survivors(B):
    """The effect the method is built on (Fig. 2a): with reward-clustered scores, the survivors
    chosen by OVF have a larger reward spread than a uniformly drawn subset of the same size -
    measured end to end on the device with the library's own diagnostics."""
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.scaled(wl.WORKLOADS["sd3"], n_groups=64, elems=256)
    inp = U.SharedInputs(w)
    table = {i: U.to_dev(wl.clustered_scores(w.n_groups, w.n_expand, w.seed, i, cluster_sigma=0.05,
                                               outlier_frac=0.15, outlier_scale=0.3, nu=3.0).reshape(-1))
             for i in (0, 1, 99)}
    spread = {}
    for selector in ("ovf", "uniform"):
        ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, torch.bfloat16)

        def lookup(i):
            ids = torch.empty(ro.n_active, device="cuda", dtype=torch.int32)
            B.rollout_traj_ids(ro.h, ids)
            return table[i][ids.long()]
        # rewards of the survivors = the stage-1 score table (the quantity the last prune saw)
        out = ro.run(U.to_dev(inp.x0), w.step_coef, w.preview_coef, lambda s, x: inp.vel_device(s, x),
                     external_scores=lookup, final_rewards=lambda: lookup(1), selector=selector)
        std = torch.empty(w.n_groups, device="cuda")
        frac = torch.empty(w.n_groups, device="cuda")
        B.group_stats(w.n_groups, w.final_keep, out.rewards, 0.5, None, std, frac)
        torch.cuda.synchronize()
        spread[selector] = (float(std.mean()), float(frac.mean()))
        assert B.rollout_status(ro.h)[0] == w.n_groups * w.final_keep
        ro.close()
    assert spread["ovf"][0] > 1.3 * spread["uniform"][0]       # larger sigma_G
    assert spread["ovf"][1] < spread["uniform"][1]             # fewer members clustered near the mean
