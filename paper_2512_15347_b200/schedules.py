"""Host-side builders of the per-step affine coefficients that the library consumes.

Every sampler step of the paper's unified SDE (Eq. unified_sde_method, Eq. euler_method) is
affine in (latent, network prediction):

    x' = c_x * x + c_v * pred + noise_std * xi          (pg_step / pg_policy_*)
    x_hat = p_x * x + p_v * pred                        (pg_score, Eq. ode_lookahead_method)

so the backbone (rectified flow or diffusion), the noise level and the time grid only enter
through (c_x, c_v, noise_std) and (p_x, p_v).  All arithmetic here is double precision Python.

Time convention (Section 5.1): index 0 is noise, the last index is data, t increases.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

StepCoef = Tuple[float, float, float]
PreviewCoef = Tuple[float, float]


# ------------------------------------------------------------------ rectified flow

def rf_drift_coef(dt: float, sigma: float) -> StepCoef:
    """Drift = the supplied prediction (b_theta = v): x' = x + v dt + sigma sqrt(dt) xi."""
    return 1.0, dt, sigma * math.sqrt(dt)


def rf_sde_coef(t: float, dt: float, sigma: float) -> StepCoef:
    """Marginal-preserving SDE of a rectified flow (Eq. rf_sde_general) with the score written
    through the velocity prediction.

    Path x_t = (1 - t) x_0 + t x_1 with x_0 ~ N(0, I) (Eq. rf_path) gives E[x_0 | x_t] = x - t v and
    grad log p_t(x) = -(x - t v) / (1 - t).  For time running from noise to data, the drift that keeps
    the marginals of dx = v dt under noise sigma dw is v + sigma^2/2 grad log p_t, hence

        b = v - sigma^2 (x - t v) / (2 (1 - t)),
        c_x = 1 - sigma^2 dt / (2 (1 - t)),   c_v = dt (1 + sigma^2 t / (2 (1 - t))).
    """
    if not 0.0 <= t < 1.0:
        raise ValueError("t must lie in [0, 1)")
    k = sigma * sigma / (2.0 * (1.0 - t))
    return 1.0 - k * dt, dt * (1.0 + k * t), sigma * math.sqrt(dt)


def rf_preview_coef(t: float) -> PreviewCoef:
    """One Euler step of the probability-flow ODE over the remaining time: x + (1 - t) v."""
    return 1.0, 1.0 - t


def uniform_times(n_steps: int) -> List[float]:
    return [s / n_steps for s in range(n_steps)]


# ------------------------------------------------------------------ diffusion (epsilon prediction)

def vp_em_coef(beta: float, sigma_bar: float, dt: float, eta: float) -> StepCoef:
    """Euler-Maruyama step of Eq. dm_sde for a variance-preserving diffusion, one step of length
    dt towards the data, with the score replaced by -eps / sigma_bar:

        f = -beta x / 2,  g^2 = beta,
        x' = x + (beta x / 2 - (1 + eta^2)/2 * beta * eps / sigma_bar) dt + eta sqrt(beta dt) xi.
    """
    if sigma_bar <= 0.0:
        raise ValueError("sigma_bar must be positive")
    return (1.0 + 0.5 * beta * dt, -0.5 * (1.0 + eta * eta) * beta * dt / sigma_bar,
            eta * math.sqrt(beta * dt))


def vp_euler_preview_coef(beta: float, sigma_bar: float, remaining: float) -> PreviewCoef:
    """Eq. ode_lookahead_method for the diffusion branch: one Euler step of the probability-flow
    drift f - g^2/2 grad log p over the remaining time."""
    return 1.0 + 0.5 * beta * remaining, -0.5 * beta * remaining / sigma_bar


def ddim_coef(alpha_t: float, sigma_t: float, alpha_next: float, sigma_next: float, eta: float) -> StepCoef:
    """Affine form of the DDIM update (Song, Meng, Ermon 2021, Eq. 12) from noise level
    (alpha_t, sigma_t) to (alpha_next, sigma_next) under the forward process of Eq. dm_forward:
        x0_hat = (x - sigma_t eps) / alpha_t,
        s      = eta * sigma_next / sigma_t * sqrt(1 - alpha_t^2 / alpha_next^2),
        x'     = alpha_next x0_hat + sqrt(sigma_next^2 - s^2) eps + s xi.
    """
    s = eta * (sigma_next / sigma_t) * math.sqrt(max(0.0, 1.0 - (alpha_t / alpha_next) ** 2))
    s = min(s, sigma_next)
    c_x = alpha_next / alpha_t
    c_v = -alpha_next * sigma_t / alpha_t + math.sqrt(max(0.0, sigma_next * sigma_next - s * s))
    return c_x, c_v, s


def x0_preview_coef(alpha_t: float, sigma_t: float) -> PreviewCoef:
    """Clean-sample estimate of an epsilon-prediction model: (x - sigma_t eps) / alpha_t."""
    return 1.0 / alpha_t, -sigma_t / alpha_t


def vp_linear_schedule(n_train: int = 1000, beta_start: float = 1e-4, beta_end: float = 2e-2):
    """(alpha_bar_t, sigma_bar_t) of the linear-beta variance-preserving schedule, t = 0..n_train-1
    (t = n_train - 1 is the noisiest)."""
    alphas, prod = [], 1.0
    for i in range(n_train):
        beta = beta_start + (beta_end - beta_start) * i / (n_train - 1)
        prod *= 1.0 - beta
        alphas.append(prod)
    return [math.sqrt(a) for a in alphas], [math.sqrt(1.0 - a) for a in alphas]


def ddim_schedule(n_steps: int, eta: float, n_train: int = 1000) -> List[StepCoef]:
    """Coefficients of an n_steps DDIM-style sampler over the linear schedule, noise first."""
    alpha, sigma = vp_linear_schedule(n_train)
    ts = [round((n_train - 1) * (1.0 - s / n_steps)) for s in range(n_steps + 1)]
    out = []
    for a, b in zip(ts[:-1], ts[1:]):
        if b <= 0:
            a_next, s_next = 1.0, 0.0
        else:
            a_next, s_next = alpha[b], sigma[b]
        out.append(ddim_coef(alpha[a], sigma[a], a_next, s_next, eta))
    return out


# ------------------------------------------------------------------ Expand-and-Prune schedules of Section 6.1

PAPER_SCHEDULES = {
    # name: (G_max, stages [(step, keep)], T)
    "pro-grpo-standard": (48, ((5, 24), (7, 12)), 10),
    "pro-grpo-flash": (24, ((5, 16), (7, 12)), 10),
    "pro-grpo-diffusion": (48, ((30, 32), (40, 8)), 50),
}


def validate_stages(n_expand: int, n_steps: int, stages: Sequence[Tuple[int, int]]) -> None:
    """Raises ValueError unless the stages form a funnel K_1 >= K_2 >= ... at increasing steps."""
    prev_step, prev_keep = -1, n_expand
    for step, keep in stages:
        if not prev_step < step < n_steps:
            raise ValueError("stage steps must increase and lie inside the step range")
        if not 1 <= keep <= prev_keep:
            raise ValueError("survivor counts must not grow")
        prev_step, prev_keep = step, keep
