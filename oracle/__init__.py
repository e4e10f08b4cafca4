"""CPU oracle of the Pro-GRPO Expand-and-Prune rollout arithmetic.

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in ``progrpo_oracle.c`` (plain C,
double precision, compiled by gcc with ``-ffp-contract=off``); this module only
builds that file, loads it through ctypes and converts numpy arrays to pointers.
``rollout`` chains the primitives in the order of the paper's Section 5.1 so that a
whole Expand-and-Prune rollout can be compared with the GPU library.

Nothing here imports, links or shares code with the CUDA package, and the CUDA
package never imports this module.  Callers: the tests, the smoke check and the
CPU-baseline leg of the benchmark.  No function is "parity unpinned": each is
checked in ``tests/test_oracle_*.py`` against known answers, closed forms, library
routines or brute force.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "progrpo_oracle.c")
_LIB = os.path.join(_HERE, "libprogrpo_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved).  Returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-Wall", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.og_num_threads.restype = ctypes.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} rejected its arguments (rc={rc})")


def num_threads() -> int:
    return int(_load().og_num_threads())


# ---------------------------------------------------------------- noise

def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    """One Philox4x32-10 block (Salmon et al., SC'11)."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().og_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return tuple(int(v) for v in out)


def philox_batch(ctr: np.ndarray, key: np.ndarray) -> np.ndarray:
    ctr = np.ascontiguousarray(ctr, dtype=np.uint32)
    key = np.ascontiguousarray(key, dtype=np.uint32)
    n = ctr.shape[0]
    assert ctr.shape == (n, 4) and key.shape == (n, 2)
    out = np.zeros((n, 4), dtype=np.uint32)
    _load().og_philox_batch(ctypes.c_int64(n), _ptr(ctr), _ptr(key), _ptr(out))
    return out


def normal_row(seed: int, step: int, trajectory: int, d: int, stream: int = 0) -> np.ndarray:
    """The d standard normals of (seed, trajectory, step); element e is entry e."""
    out = np.zeros(d, dtype=np.float64)
    rc = _load().og_normal_row(ctypes.c_uint64(seed), ctypes.c_uint32(step),
                               ctypes.c_uint32(trajectory), ctypes.c_uint32(stream),
                               ctypes.c_int64(d), _ptr(out))
    _check(rc, "normal_row")
    return out


# ---------------------------------------------------------------- inputs

def _vel_arg(vel: np.ndarray):
    """fp32 array -> (ptr, 0); uint16 array of bf16 bit patterns -> (ptr, 1)."""
    if vel.dtype == np.float32:
        return np.ascontiguousarray(vel), 0
    if vel.dtype == np.uint16:
        return np.ascontiguousarray(vel), 1
    raise TypeError("velocity must be float32 or uint16 (bf16 bit patterns)")


# ---------------------------------------------------------------- primitives

def step(x_in: np.ndarray, vel: np.ndarray, traj_id: np.ndarray, seed: int, step_index: int,
         c_x: float, c_v: float, noise_std: float, src_slot: Optional[np.ndarray] = None,
         logp_mean: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Euler-Maruyama update and Gaussian policy log-prob (Eq. euler_method).

    Returns (x_out fp32 [n, d], logp fp64 [n]); n = len(traj_id).
    """
    x_in = np.ascontiguousarray(x_in, dtype=np.float32)
    vel, vdt = _vel_arg(vel)
    traj_id = np.ascontiguousarray(traj_id, dtype=np.int32)
    n = traj_id.shape[0]
    d = x_in.shape[1]
    if src_slot is not None:
        src_slot = np.ascontiguousarray(src_slot, dtype=np.int32)
        assert src_slot.shape[0] == n
        assert src_slot.min(initial=0) >= 0 and src_slot.max(initial=0) < x_in.shape[0]
    else:
        assert x_in.shape[0] >= n
    assert vel.shape == x_in.shape
    x_out = np.empty((n, d), dtype=np.float32)
    logp = np.empty(n, dtype=np.float64)
    rc = _load().og_step(ctypes.c_int64(n), ctypes.c_int64(d), _ptr(x_in), _ptr(vel),
                         ctypes.c_int(vdt), _ptr(src_slot), _ptr(traj_id),
                         ctypes.c_uint64(seed), ctypes.c_uint32(step_index),
                         ctypes.c_double(c_x), ctypes.c_double(c_v), ctypes.c_double(noise_std),
                         ctypes.c_int(1 if logp_mean else 0), _ptr(x_out), _ptr(logp))
    _check(rc, "step")
    return x_out, logp


def transition_logp(x_in: np.ndarray, vel: np.ndarray, x_next: np.ndarray, c_x: float,
                    c_v: float, noise_std: float, logp_mean: bool = False) -> np.ndarray:
    x_in = np.ascontiguousarray(x_in, dtype=np.float32)
    vel, vdt = _vel_arg(vel)
    x_next = np.ascontiguousarray(x_next, dtype=np.float64)
    n, d = x_in.shape
    out = np.empty(n, dtype=np.float64)
    rc = _load().og_transition_logp(ctypes.c_int64(n), ctypes.c_int64(d), _ptr(x_in), _ptr(vel),
                                    ctypes.c_int(vdt), _ptr(x_next), ctypes.c_double(c_x),
                                    ctypes.c_double(c_v), ctypes.c_double(noise_std),
                                    ctypes.c_int(1 if logp_mean else 0), _ptr(out))
    _check(rc, "transition_logp")
    return out


def score(x: np.ndarray, vel: np.ndarray, p_x: float, p_v: float,
          want_preview: bool = False) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """ODE look-ahead preview (Eq. ode_lookahead_method) and its mean as latent score."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    vel, vdt = _vel_arg(vel)
    n, d = x.shape
    assert vel.shape == x.shape
    out = np.empty(n, dtype=np.float64)
    prev = np.empty((n, d), dtype=np.float32) if want_preview else None
    rc = _load().og_score(ctypes.c_int64(n), ctypes.c_int64(d), _ptr(x), _ptr(vel),
                          ctypes.c_int(vdt), ctypes.c_double(p_x), ctypes.c_double(p_v),
                          _ptr(out), _ptr(prev))
    _check(rc, "score")
    return out, prev


def ovf_exhaustive(scores: np.ndarray, k: int) -> Tuple[float, np.ndarray]:
    """Max-variance k-subset by enumeration (Eq. ovf); n <= 24."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    n = scores.shape[0]
    subset = np.zeros(k, dtype=np.int32)
    var = ctypes.c_double(0.0)
    rc = _load().og_ovf_exhaustive(ctypes.c_int(n), ctypes.c_int(k), _ptr(scores), _ptr(subset),
                                   ctypes.byref(var))
    _check(rc, "ovf_exhaustive")
    return float(var.value), subset


def ovf_select(scores: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """OVF for [G, n] (or [n]) fp32 scores.  Returns (keep_idx int32 [G, k], sel_var [G])."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    squeeze = scores.ndim == 1
    s2 = scores.reshape(1, -1) if squeeze else scores
    g, n = s2.shape
    keep = np.zeros((g, k), dtype=np.int32)
    var = np.zeros(g, dtype=np.float64)
    rc = _load().og_ovf_select_groups(ctypes.c_int(g), ctypes.c_int(n), ctypes.c_int(k), _ptr(s2),
                                      _ptr(keep), _ptr(var))
    _check(rc, "ovf_select")
    return (keep[0], var[0:1]) if squeeze else (keep, var)


def compact_rows(keep_idx: np.ndarray, src: np.ndarray, n_prev: int) -> np.ndarray:
    """Gather the kept rows of every group, ascending slot order."""
    keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
    g, k = keep_idx.shape
    src = np.ascontiguousarray(src)
    assert src.shape[0] == g * n_prev
    row_bytes = src.dtype.itemsize * int(np.prod(src.shape[1:], dtype=np.int64))
    dst = np.empty((g * k,) + src.shape[1:], dtype=src.dtype)
    rc = _load().og_compact_rows(ctypes.c_int(g), ctypes.c_int(n_prev), ctypes.c_int(k),
                                 _ptr(keep_idx), _ptr(src), _ptr(dst), ctypes.c_size_t(row_bytes))
    _check(rc, "compact_rows")
    return dst


def advantages(rewards: np.ndarray, eps: float) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Group-relative advantages (Eq. advantage / Eq. advK) for [G, K] rewards."""
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    g, k = rewards.shape
    adv = np.empty((g, k), dtype=np.float64)
    mean = np.empty(g, dtype=np.float64)
    std = np.empty(g, dtype=np.float64)
    rc = _load().og_advantages(ctypes.c_int(g), ctypes.c_int(k), _ptr(rewards),
                               ctypes.c_double(eps), _ptr(adv), _ptr(mean), _ptr(std))
    _check(rc, "advantages")
    return adv, mean, std


# ---------------------------------------------------------------- whole rollout

@dataclass
class RolloutResult:
    x_final: np.ndarray                       # [G*K, d] fp32
    logp: List[np.ndarray]                    # per step, fp64 [n_active at that step]
    traj_id: np.ndarray                       # [G*K] original trajectory ids of survivors
    stage_scores: List[np.ndarray] = field(default_factory=list)   # per stage [G, K_i] fp32
    stage_keep: List[np.ndarray] = field(default_factory=list)     # per stage [G, k] int32
    stage_var: List[np.ndarray] = field(default_factory=list)
    rewards: Optional[np.ndarray] = None      # [G, K] fp32
    adv: Optional[np.ndarray] = None
    mean: Optional[np.ndarray] = None
    std: Optional[np.ndarray] = None
    x_steps: Optional[List[np.ndarray]] = None


def rollout(x0: np.ndarray, n_groups: int, n_expand: int, n_steps: int,
            stages: Sequence[Tuple[int, int]], seed: int,
            step_coef: Callable[[int], Tuple[float, float, float]],
            preview_coef: Callable[[int], Tuple[float, float]],
            velocity: Callable[[int, np.ndarray, np.ndarray], np.ndarray],
            external_scores: Optional[Callable[[int, np.ndarray], np.ndarray]] = None,
            final_rewards: Optional[Callable[[np.ndarray, np.ndarray], np.ndarray]] = None,
            adv_eps: float = 1e-6, group_offset: int = 0, keep_steps: bool = False) -> RolloutResult:
    """Expand-and-Prune rollout in the order of Section 5.1 / 5.2.

    For every step s: obtain the prediction v(x_s, t_s) for the active rows; if s is a
    checkpoint, score the previews, run OVF per group and keep only the survivors (they
    are the only rows that take step s and later steps); then take the SDE step.
    Finally compute group-relative advantages over the survivors' rewards.

    ``velocity(step, x_active, traj_id)`` returns fp32 or uint16(bf16) [n_active, d];
    ``external_scores(stage, traj_id)`` (optional) returns fp32 [n_active] and replaces
    the preview mean; ``final_rewards(x_final, traj_id)`` returns fp32 [n_active]
    (default: mean of the final latent).
    """
    x = np.ascontiguousarray(x0, dtype=np.float32)
    k_cur = n_expand
    assert x.shape[0] == n_groups * n_expand
    traj = (np.arange(n_groups * n_expand, dtype=np.int64)
            + group_offset * n_expand).astype(np.int32)
    res = RolloutResult(x_final=x, logp=[], traj_id=traj, x_steps=[] if keep_steps else None)
    stage_at = {int(s): (i, int(k)) for i, (s, k) in enumerate(stages)}
    for s in range(n_steps):
        vel = velocity(s, x, traj)
        src = None
        if s in stage_at:
            si, k = stage_at[s]
            if external_scores is not None:
                sc32 = np.asarray(external_scores(si, traj), dtype=np.float32)
            else:
                p_x, p_v = preview_coef(s)
                sc, _ = score(x, vel, p_x, p_v)
                sc32 = sc.astype(np.float32)
            sc32 = sc32.reshape(n_groups, k_cur)
            keep, var = ovf_select(sc32, k)
            res.stage_scores.append(sc32)
            res.stage_keep.append(keep)
            res.stage_var.append(var)
            src = (keep + (np.arange(n_groups, dtype=np.int32) * k_cur)[:, None]).reshape(-1)
            src = src.astype(np.int32)
            traj = compact_rows(keep, traj.reshape(-1, 1), k_cur).reshape(-1)
            k_cur = k
        c_x, c_v, ns = step_coef(s)
        x, lp = step(x, vel, traj, seed, s, c_x, c_v, ns, src_slot=src)
        res.logp.append(lp)
        if keep_steps:
            res.x_steps.append(x)
    res.x_final = x
    res.traj_id = traj
    if final_rewards is not None:
        rw = np.asarray(final_rewards(x, traj), dtype=np.float32)
    else:
        rw = x.astype(np.float64).mean(axis=1).astype(np.float32)
    rw = rw.reshape(n_groups, k_cur)
    res.rewards = rw
    res.adv, res.mean, res.std = advantages(rw, adv_eps)
    return res


def survivor_rows(n_groups: int, n_expand: int, n_steps: int, stages: Sequence[Tuple[int, int]],
                  stage_keep: Sequence[np.ndarray]) -> np.ndarray:
    """Where the final survivors sat at every step (Section 5.1; Eq. pro_grpo_method sums over the
    survivors only, but over all T steps, so their log-probs and latents from before a prune must
    be found among the rows that were active then).

    Written as the definition: every group carries the list of original slots of its active rows
    through the schedule (a prune at step s replaces the list by its kept entries, in ascending
    slot order, before step s is taken); afterwards every final survivor is looked up by identity
    in each step's list.  stage_keep[i] is the [G, k_i] slot list of stage i.  Returns int32
    [T, G*K]: rows[t][g*K + j] = row (group-major among the rows active at step t) of the j-th
    final survivor of group g.
    """
    stage_at = {int(s): i for i, (s, _) in enumerate(stages)}
    active = [list(range(n_expand)) for _ in range(n_groups)]
    per_step = []
    for t in range(n_steps):
        if t in stage_at:
            keep = np.asarray(stage_keep[stage_at[t]]).reshape(n_groups, -1)
            active = [[active[g][int(i)] for i in keep[g]] for g in range(n_groups)]
        per_step.append([list(a) for a in active])
    k_final = len(active[0])
    rows = np.empty((n_steps, n_groups * k_final), dtype=np.int32)
    for t in range(n_steps):
        k_t = len(per_step[t][0])
        for g in range(n_groups):
            for j, orig in enumerate(active[g]):
                rows[t, g * k_final + j] = g * k_t + per_step[t][g].index(orig)
    return rows


# ---------------------------------------------------------------- policy update (Eq. ratio_method, Eq. pro_grpo_method)

def policy_logprob(x: np.ndarray, x_next: np.ndarray, vel: np.ndarray, vel_ref: Optional[np.ndarray],
                   c_x: float, c_v: float, noise_std: float, logp_mean: bool = False):
    """log pi_theta of the stored transitions under a new prediction, and KL to a reference."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    x_next = np.ascontiguousarray(x_next, dtype=np.float32)
    vel, vdt = _vel_arg(vel)
    n, d = x.shape
    logp = np.empty(n, dtype=np.float64)
    kl = None
    if vel_ref is not None:
        vel_ref, vdt2 = _vel_arg(vel_ref)
        assert vdt2 == vdt
        kl = np.empty(n, dtype=np.float64)
    rc = _load().og_policy_logprob(ctypes.c_int64(n), ctypes.c_int64(d), _ptr(x), _ptr(x_next), _ptr(vel),
                                   _ptr(vel_ref), ctypes.c_int(vdt), ctypes.c_double(c_x),
                                   ctypes.c_double(c_v), ctypes.c_double(noise_std),
                                   ctypes.c_int(1 if logp_mean else 0), _ptr(logp), _ptr(kl))
    _check(rc, "policy_logprob")
    return logp, kl


def policy_objective(logp_new: np.ndarray, logp_old: np.ndarray, kl: Optional[np.ndarray],
                     adv: np.ndarray, clip_eps: float, beta: float):
    """Clipped surrogate objective, ratios and dJ/dlogp_new for [T, n] log-probs."""
    logp_new = np.ascontiguousarray(logp_new, dtype=np.float64)
    logp_old = np.ascontiguousarray(logp_old, dtype=np.float64)
    adv = np.ascontiguousarray(adv, dtype=np.float64)
    T, n = logp_new.shape
    assert logp_old.shape == (T, n) and adv.shape == (n,)
    if kl is not None:
        kl = np.ascontiguousarray(kl, dtype=np.float64)
        assert kl.shape == (T, n)
    ratio = np.empty((T, n), dtype=np.float64)
    dlogp = np.empty((T, n), dtype=np.float64)
    obj = ctypes.c_double(0.0)
    rc = _load().og_policy_objective(ctypes.c_int64(T), ctypes.c_int64(n), _ptr(logp_new), _ptr(logp_old),
                                     _ptr(kl), _ptr(adv), ctypes.c_double(clip_eps), ctypes.c_double(beta),
                                     _ptr(ratio), _ptr(dlogp), ctypes.byref(obj))
    _check(rc, "policy_objective")
    return float(obj.value), ratio, dlogp


def policy_backward(x: np.ndarray, x_next: np.ndarray, vel: np.ndarray, vel_ref: Optional[np.ndarray],
                    c_x: float, c_v: float, noise_std: float, dlogp: np.ndarray, dkl: float,
                    logp_mean: bool = False) -> np.ndarray:
    """dJ/dvel for one step (fp64 [n, d])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    x_next = np.ascontiguousarray(x_next, dtype=np.float32)
    vel, vdt = _vel_arg(vel)
    if vel_ref is not None:
        vel_ref, _ = _vel_arg(vel_ref)
    dlogp = np.ascontiguousarray(dlogp, dtype=np.float64)
    n, d = x.shape
    grad = np.empty((n, d), dtype=np.float64)
    rc = _load().og_policy_backward(ctypes.c_int64(n), ctypes.c_int64(d), _ptr(x), _ptr(x_next), _ptr(vel),
                                    _ptr(vel_ref), ctypes.c_int(vdt), ctypes.c_double(c_x),
                                    ctypes.c_double(c_v), ctypes.c_double(noise_std),
                                    ctypes.c_int(1 if logp_mean else 0), _ptr(dlogp), ctypes.c_double(dkl),
                                    _ptr(grad))
    _check(rc, "policy_backward")
    return grad


# ---------------------------------------------------------------- diagnostics / uniform baseline

def group_stats(scores: np.ndarray, delta: float):
    """(mean, population std, fraction inside |R - mu| <= delta sigma) per group of [G, n] scores."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    g, n = scores.shape
    mean = np.empty(g)
    std = np.empty(g)
    frac = np.empty(g)
    rc = _load().og_group_stats(ctypes.c_int(g), ctypes.c_int(n), _ptr(scores), ctypes.c_double(delta),
                                _ptr(mean), _ptr(std), _ptr(frac))
    _check(rc, "group_stats")
    return mean, std, frac


def select_uniform(n_groups: int, n: int, k: int, seed: int, stage: int, group_offset: int = 0) -> np.ndarray:
    """Reproducible uniform k-of-n subsampling per group; int32 [G, k], ascending slots."""
    keep = np.zeros((n_groups, k), dtype=np.int32)
    rc = _load().og_select_uniform(ctypes.c_int(n_groups), ctypes.c_int(n), ctypes.c_int(k),
                                   ctypes.c_uint64(seed), ctypes.c_uint32(stage),
                                   ctypes.c_uint32(group_offset), _ptr(keep))
    _check(rc, "select_uniform")
    return keep
