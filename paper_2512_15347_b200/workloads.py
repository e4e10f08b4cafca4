"""Seeded synthetic inputs and the five workload shapes.

This module produces *inputs only* (initial latents, stand-in network predictions,
stand-in reward-model scores, per-step schedule coefficients).  It contains none of the
rollout arithmetic and imports neither the CUDA binding nor any checker, so the GPU
library and an independent CPU check can both be fed the very same arrays.

The denoiser, VAE decoder and reward model of the paper are not available; their
outputs are replaced by seeded random tensors with the shapes of the paper's
workloads (Stable-Diffusion style 4x32x32 / 4x64x64 latents, SD3 / FLUX style
16x128x128 latents; group schedules such as 48->24->12 from the experimental
settings of Section 6.1).
"""
from __future__ import annotations

import dataclasses
import functools
import math
from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from . import schedules as sch


@dataclass(frozen=True)
class Workload:
    name: str
    n_groups: int                 # G prompt groups
    n_expand: int                 # N0 = G_max trajectories per group
    stages: Tuple[Tuple[int, int], ...]   # (step index, survivors per group)
    n_steps: int                  # T
    elems: int                    # d = C*H*W
    channels: int
    vel_dtype: str                # "fp32" | "bf16"
    seed: int
    velocity: str                 # "affine" (config 1) | "normal" (fresh N(0,1) per step) | "eps"
    scores: str                   # "preview" | "external"
    sigma: float = 0.7            # noise_std = sigma * sqrt(dt)
    adv_eps: float = 1e-6
    coef: str = "rf-drift"        # source of the per-step coefficients, see step_coef()
    eta: float = 1.0              # stochasticity of the diffusion samplers ("ddim", "vp-em")

    @property
    def final_keep(self) -> int:
        return self.stages[-1][1] if self.stages else self.n_expand

    def active_at(self, step: int) -> int:
        """Trajectories per group that take SDE step `step` (pruning precedes the step)."""
        k = self.n_expand
        for s, keep in self.stages:
            if step >= s:
                k = keep
        return k

    def rows_before(self, step: int) -> int:
        """Trajectories per group alive when the prediction for `step` is made."""
        k = self.n_expand
        for s, keep in self.stages:
            if step > s:
                k = keep
        return k

    @property
    def traj_steps(self) -> int:
        return sum(self.n_groups * self.active_at(s) for s in range(self.n_steps))

    @property
    def element_steps(self) -> int:
        return self.traj_steps * self.elems

    @property
    def score_rows(self) -> int:
        """Rows scored from (x, v) over all stages (0 for external scores)."""
        if self.scores != "preview":
            return 0
        return sum(self.n_groups * self.rows_before(s) for s, _ in self.stages)

    def step_coef(self, step: int) -> Tuple[float, float, float]:
        """(c_x, c_v, noise_std) of SDE step `step` on the uniform grid t_s = s/T.

        coef = "rf-drift": drift = the supplied prediction (c_x = 1, c_v = dt);
        "rf-sde": rectified flow with the score-corrected drift of Eq. rf_sde_general;
        "ddim": epsilon-prediction diffusion, the T-step DDIM / ancestral sampler (stochasticity
        eta) over the 1000-step linear-beta schedule; its last step lands on the clean sample and
        is deterministic (noise_std = 0);
        "vp-em": Euler-Maruyama of Eq. dm_sde for the continuous variance-preserving diffusion
        with beta(tau) = 0.1 + 19.9 tau, tau = 1 - s/T the noise-level time."""
        dt = 1.0 / self.n_steps
        if self.coef == "rf-drift":
            return sch.rf_drift_coef(dt, self.sigma)
        if self.coef == "rf-sde":
            return sch.rf_sde_coef(step * dt, dt, self.sigma)
        if self.coef == "ddim":
            return _ddim_table(self.n_steps, self.eta)[step]
        if self.coef == "vp-em":
            beta, sigma_bar = _vp_continuous(1.0 - step * dt)
            return sch.vp_em_coef(beta, sigma_bar, dt, self.eta)
        raise ValueError(f"unknown coefficient source {self.coef!r}")

    def preview_coef(self, step: int) -> Tuple[float, float]:
        """(p_x, p_v) of the look-ahead preview at step `step` (Eq. ode_lookahead_method): one Euler
        step of the probability-flow ODE over the remaining time for the rectified-flow sources and
        "vp-em", the clean-sample estimate (x - sigma_t eps) / alpha_t for "ddim"."""
        t = step / self.n_steps
        if self.coef in ("rf-drift", "rf-sde"):
            return sch.rf_preview_coef(t)
        if self.coef == "ddim":
            alpha, sigma = _vp_table()
            i = round((len(alpha) - 1) * (1.0 - t))
            return sch.x0_preview_coef(alpha[i], sigma[i])
        if self.coef == "vp-em":
            beta, sigma_bar = _vp_continuous(1.0 - t)
            return sch.vp_euler_preview_coef(beta, sigma_bar, 1.0 - t)
        raise ValueError(f"unknown coefficient source {self.coef!r}")


@functools.lru_cache(maxsize=None)
def _vp_table():
    return sch.vp_linear_schedule()


@functools.lru_cache(maxsize=None)
def _ddim_table(n_steps: int, eta: float):
    return sch.ddim_schedule(n_steps, eta)


def _vp_continuous(tau: float) -> Tuple[float, float]:
    """(beta(tau), sigma_bar(tau)) of the continuous linear-beta variance-preserving diffusion."""
    b0, b1 = 0.1, 20.0
    integral = b0 * tau + 0.5 * (b1 - b0) * tau * tau
    return b0 + (b1 - b0) * tau, math.sqrt(-math.expm1(-integral))


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, 16, ((3, 8),), 10, 4 * 32 * 32, 4, "fp32", 0, "affine", "preview"),
    "sd15": Workload("sd15", 8, 24, ((4, 12),), 20, 4 * 64 * 64, 4, "bf16", 1, "normal", "preview"),
    "sd3": Workload("sd3", 16, 48, ((3, 24), (6, 12)), 28, 16 * 128 * 128, 16, "bf16", 3,
                    "normal", "external"),
    "large": Workload("large", 64, 64, ((2, 32), (5, 16), (8, 16)), 28, 16 * 128 * 128, 16, "bf16",
                      7, "normal", "preview"),
    # the schedules of the paper's experimental settings (Section 6.1), 16 prompt groups each:
    # Standard 48 -> 24 -> 12 and Flash 24 -> 16 -> 12 at steps {5, 7} of 10 on SD3-sized latents,
    # and 48 -> 32 -> 8 at steps {30, 40} of 50 on SD-v1.4-sized latents
    "pro-standard": Workload("pro-standard", 16, 48, ((5, 24), (7, 12)), 10, 16 * 128 * 128, 16, "bf16",
                             11, "normal", "preview"),
    "pro-flash": Workload("pro-flash", 16, 24, ((5, 16), (7, 12)), 10, 16 * 128 * 128, 16, "bf16",
                          12, "normal", "preview"),
    # (epsilon-prediction diffusion backbone: DDIM / ancestral coefficients, clean-sample preview,
    # predictions correlated with the latent as a noise-prediction network's are)
    "pro-diffusion": Workload("pro-diffusion", 16, 48, ((30, 32), (40, 8)), 50, 4 * 64 * 64, 4, "fp32",
                              13, "eps", "preview", coef="ddim", eta=1.0),
}

def workload_to_dict(w: Workload) -> dict:
    d = dataclasses.asdict(w)
    d["stages"] = [list(st) for st in w.stages]
    return d


def workload_from_dict(d: dict) -> Workload:
    """A workload from its JSON form (the files under configs/ mirror the built-in ones; a caller
    can describe its own batch shape and schedule the same way)."""
    d = dict(d)
    d["stages"] = tuple((int(s), int(k)) for s, k in d.get("stages", ()))
    unknown = set(d) - {f.name for f in dataclasses.fields(Workload)}
    if unknown:
        raise ValueError(f"unknown workload fields: {sorted(unknown)}")
    w = Workload(**d)
    sch.validate_stages(w.n_expand, w.n_steps, w.stages)
    if w.elems % 4 or w.elems < 4 or w.vel_dtype not in ("fp32", "bf16"):
        raise ValueError("elems must be a positive multiple of 4 and vel_dtype fp32 or bf16")
    return w


def load_workload(path: str) -> Workload:
    import json
    with open(path) as f:
        return workload_from_dict(json.load(f))


# OVF selection microbenchmark: 4096 groups x 256 scores, keep 32.
OVF_MICRO = dict(n_groups=4096, n=256, k=32, seed=4)


def scaled(w: Workload, *, n_groups: Optional[int] = None, elems: Optional[int] = None,
           name: Optional[str] = None) -> Workload:
    """A smaller copy of a workload (fewer groups and/or shorter latents) for quick checks."""
    from dataclasses import replace
    return replace(w, n_groups=n_groups or w.n_groups, elems=elems or w.elems,
                   name=name or (w.name + "-scaled"))


def _gen(device, *words: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for w in words:
        s = (s ^ (int(w) + 0x632BE59BD9B4E019)) * 0xD1342543DE82EF95 % (1 << 63)
    g.manual_seed(s)
    return g


def initial_latents(w: Workload, device="cpu") -> torch.Tensor:
    """x_0 ~ N(0, I), fp32 [G*N0, d]."""
    return torch.randn(w.n_groups * w.n_expand, w.elems, generator=_gen(device, w.seed, 101),
                       device=device, dtype=torch.float32)


def normal_velocity(w: Workload, step: int, rows: int, device="cpu") -> torch.Tensor:
    """Stand-in network prediction for one step: fresh N(0,1), in the workload's dtype."""
    v = normal_noise(w, step, rows, device)
    return v.to(torch.bfloat16) if w.vel_dtype == "bf16" else v


def normal_noise(w: Workload, step: int, rows: int, device="cpu") -> torch.Tensor:
    """The fp32 N(0,1) draws behind normal_velocity (before any rounding to bf16)."""
    return torch.randn(rows, w.elems, generator=_gen(device, w.seed, 202, step), device=device,
                       dtype=torch.float32)


def eps_mix(w: Workload, step: int) -> Tuple[float, float]:
    """(a, b) of the stand-in noise-prediction network at step `step`: eps_hat = a x + b z.

    For unit-variance Gaussian data under x_t = alpha_t x_1 + sigma_t eps the exact noise
    prediction is E[eps | x_t] = sigma_t x_t; the stand-in adds an independent error term
    alpha_t z, z ~ N(0, I), so that eps_hat is N(0, 1) per element like the target and correlated
    with the latent like a real network's output (an uncorrelated prediction would let the
    epsilon-prediction samplers, whose c_x exceeds 1, blow the latents up)."""
    t = step / w.n_steps
    if w.coef == "ddim":
        alpha, sigma = _vp_table()
        i = round((len(alpha) - 1) * (1.0 - t))
        return sigma[i], alpha[i]
    _, sigma_bar = _vp_continuous(1.0 - t)
    return sigma_bar, math.sqrt(max(0.0, 1.0 - sigma_bar * sigma_bar))


def eps_velocity(x: torch.Tensor, z: torch.Tensor, a: float, b: float, vel_dtype: str) -> torch.Tensor:
    """eps_hat = a x + b z as three separately rounded fp32 operations (identical on CPU and GPU),
    then rounded to the workload's prediction dtype."""
    v = x * a
    v += z * b
    return v.to(torch.bfloat16) if vel_dtype == "bf16" else v


def affine_field(w: Workload, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Per-channel (a_c, b_c) with a_c ~ U(-1, 0), b_c ~ N(0, 0.1^2), expanded to [d]."""
    g = _gen("cpu", w.seed, 303)
    a = -torch.rand(w.channels, generator=g, dtype=torch.float32)
    b = 0.1 * torch.randn(w.channels, generator=g, dtype=torch.float32)
    per = w.elems // w.channels
    return (a.repeat_interleave(per).to(device), b.repeat_interleave(per).to(device))


def affine_velocity(x: torch.Tensor, a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """v = a_c * x + b_c as two separately rounded fp32 operations (identical on CPU and GPU)."""
    v = x * a
    v += b
    return v


def _student_t(rng: np.random.Generator, nu: float, size) -> np.ndarray:
    return rng.standard_t(nu, size=size)


def clustered_scores(n_groups: int, n: int, seed: int, stage: int, *, cluster_sigma: float,
                     outlier_frac: float, outlier_scale: float, nu: float) -> np.ndarray:
    """Reward-clustered stand-in scores, fp32 [G, n].

    Each group has a mean mu_g ~ U(0,1); a score is mu_g + cluster_sigma*z with probability
    1 - outlier_frac and mu_g + outlier_scale*t_nu otherwise (heavy-tailed outliers).
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, 1000 + stage]))
    mu = rng.random((n_groups, 1))
    z = rng.standard_normal((n_groups, n))
    t = _student_t(rng, nu, (n_groups, n))
    outlier = rng.random((n_groups, n)) < outlier_frac
    return (mu + np.where(outlier, outlier_scale * t, cluster_sigma * z)).astype(np.float32)


def sd3_stage_scores(w: Workload, stage: int, traj_id: np.ndarray) -> np.ndarray:
    """External scores for the SD3-shaped workload, keyed by original trajectory and stage.

    A full [G, N0] table is drawn per stage; the entries of the still-active trajectories
    are returned in their current (compacted) order.
    """
    table = clustered_scores(w.n_groups, w.n_expand, w.seed, stage, cluster_sigma=0.05,
                             outlier_frac=0.15, outlier_scale=0.3, nu=3.0).reshape(-1)
    return table[np.asarray(traj_id, dtype=np.int64)]


def ovf_micro_scores(n_groups: int = OVF_MICRO["n_groups"], n: int = OVF_MICRO["n"],
                     seed: int = OVF_MICRO["seed"]) -> np.ndarray:
    """Scores of the OVF microbenchmark: 80 % N(mu_g, 0.02), 20 % Student-t(2) scaled 0.3."""
    return clustered_scores(n_groups, n, seed, 0, cluster_sigma=0.02, outlier_frac=0.2,
                            outlier_scale=0.3, nu=2.0)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (CPU) -> numpy uint16 bit patterns."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def as_numpy_velocity(v: torch.Tensor) -> np.ndarray:
    v = v.detach().cpu()
    return bf16_bits(v) if v.dtype == torch.bfloat16 else v.numpy()
