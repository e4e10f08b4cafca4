"""ctypes binding of libprogrpo.so: same names as the C ABI (minus the ``pg_`` prefix),
argument marshalling only.  Tensors are torch CUDA tensors (or raw integer addresses); every
computation happens inside the library's kernels.  There is no fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprogrpo.so")

OK, EINVAL, ESTATE, ECUDA, ENONFINITE, ETIMEOUT, ENOMEM, ECAPACITY, EINDEX, EDEVICE = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9
STATIC_MAX_ROWS, STATIC_MAX_PARTIALS = 8192, 65536
VEL_F32, VEL_BF16 = 0, 1
MAX_GROUP = 1024


class PgError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = lib().pg_strerror(code).decode()
        extra = f" (cudaError {lib().pg_last_cuda_error()})" if code == ECUDA else ""
        super().__init__(f"{what}: {msg}{extra}")


class Config(ctypes.Structure):
    _fields_ = [("n_groups", ctypes.c_int32), ("n_expand", ctypes.c_int32),
                ("elems", ctypes.c_int32), ("n_steps", ctypes.c_int32),
                ("n_stages", ctypes.c_int32),
                ("stage_step", ctypes.POINTER(ctypes.c_int32)),
                ("stage_keep", ctypes.POINTER(ctypes.c_int32)),
                ("seed", ctypes.c_uint64), ("group_offset", ctypes.c_int32),
                ("vel_dtype", ctypes.c_int32), ("logp_mean", ctypes.c_int32),
                ("adv_eps", ctypes.c_float)]


class StepCoef(ctypes.Structure):
    _fields_ = [("c_x", ctypes.c_double), ("c_v", ctypes.c_double), ("noise_std", ctypes.c_double)]


class RolloutOutputs(ctypes.Structure):
    _fields_ = [("x_final", ctypes.c_void_p), ("logp", ctypes.c_void_p), ("keep_idx", ctypes.c_void_p),
                ("adv", ctypes.c_void_p), ("rewards", ctypes.c_void_p), ("traj_id", ctypes.c_void_p),
                ("n_final", ctypes.c_int32), ("n_logp", ctypes.c_int64), ("n_keep", ctypes.c_int64)]


class PreviewCoef(ctypes.Structure):
    _fields_ = [("p_x", ctypes.c_double), ("p_v", ctypes.c_double)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the library (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2512_15347_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64,
                             ctypes.c_size_t)
    L.pg_rollout_init.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(vp)]
    L.pg_rollout_destroy.argtypes = [vp]
    L.pg_rollout_reset.argtypes = [vp, vp]
    L.pg_rollout_restore.argtypes = [vp, i32, i32, vp, vp]
    L.pg_rollout_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.pg_step.argtypes = [vp, i32, ctypes.POINTER(StepCoef), vp, vp, vp, vp, vp, vp]
    L.pg_step_reward.argtypes = [vp, i32, ctypes.POINTER(StepCoef), vp, vp, vp, vp, vp, vp, vp]
    L.pg_score.argtypes = [vp, ctypes.POINTER(PreviewCoef), vp, vp, vp, vp, vp]
    L.pg_preview.argtypes = [vp, ctypes.POINTER(PreviewCoef), vp, vp, vp, i32, vp]
    L.pg_score_preview.argtypes = [vp, ctypes.POINTER(PreviewCoef), vp, vp, vp, vp, i32, vp]
    L.pg_prune_ovf.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    L.pg_prune_uniform.argtypes = [vp, i32, vp, vp, vp]
    L.pg_group_stats.argtypes = [i32, i32, vp, ctypes.c_float, vp, vp, vp, vp]
    L.pg_compact.argtypes = [vp, vp, vp, vp, sz, vp]
    L.pg_advantages.argtypes = [vp, vp, vp, vp, vp, vp]
    L.pg_policy_logprob.argtypes = [vp, ctypes.POINTER(StepCoef), vp, vp, vp, vp, vp, vp, vp]
    L.pg_policy_objective.argtypes = [vp, i32, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, vp, vp, vp]
    L.pg_policy_backward.argtypes = [vp, ctypes.POINTER(StepCoef), vp, vp, vp, vp, vp, ctypes.c_double, vp, vp]
    L.pg_ovf_select_batched.argtypes = [i32, i32, i32, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    L.pg_rollout_host_workspace_bytes.argtypes = [ctypes.POINTER(Config)]
    L.pg_rollout_host_workspace_bytes.restype = sz
    L.pg_rollout_host.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(StepCoef),
                                  ctypes.POINTER(PreviewCoef), vp, ctypes.POINTER(vp),
                                  ctypes.POINTER(vp), vp, vp, vp, vp, vp, vp, vp, sz]
    L.pg_rollout_host_on.argtypes = [vp, ctypes.POINTER(StepCoef), ctypes.POINTER(PreviewCoef), vp,
                                     ctypes.POINTER(vp), ctypes.POINTER(vp), vp, vp, vp, vp, vp, vp, vp, sz]
    L.pg_score_static.argtypes = [i32, i32, i32, ctypes.POINTER(PreviewCoef), vp, vp, vp, vp]
    L.pg_rollout_run_workspace_bytes.argtypes = [ctypes.POINTER(Config)]
    L.pg_rollout_run_workspace_bytes.restype = sz
    L.pg_rollout_run.argtypes = [vp, ctypes.POINTER(StepCoef), ctypes.POINTER(PreviewCoef), vp,
                                 ctypes.POINTER(vp), ctypes.POINTER(vp), vp, vp, sz,
                                 ctypes.POINTER(RolloutOutputs), vp]
    L.pg_rollout_traj_ids.argtypes = [vp, vp, vp]
    L.pg_selftest_bounded_wait.argtypes = [vp, vp]
    L.pg_survivor_rows.argtypes = [vp, vp, vp, vp]
    L.pg_survivor_logp.argtypes = [vp, vp, vp, vp, vp]
    L.pg_gather_rows.argtypes = [vp, vp, i32, i32, vp, vp, sz, vp]
    L.pg_philox_raw.argtypes = [i64, vp, vp, vp, vp]
    L.pg_normal_rows.argtypes = [u64, i32, i32, i32, i32, vp, vp, vp]
    L.pg_strerror.argtypes = [ctypes.c_int]
    L.pg_strerror.restype = ctypes.c_char_p
    L.pg_last_cuda_error.restype = ctypes.c_int
    L.pg_launch_count.restype = ctypes.c_uint64
    for name in ("pg_rollout_init", "pg_rollout_destroy", "pg_rollout_reset", "pg_rollout_status",
                 "pg_step", "pg_score", "pg_prune_ovf", "pg_compact", "pg_advantages",
                 "pg_ovf_select_batched", "pg_rollout_host", "pg_rollout_traj_ids",
                 "pg_philox_raw", "pg_normal_rows", "pg_score_static", "pg_policy_logprob",
                 "pg_policy_objective", "pg_policy_backward", "pg_prune_uniform", "pg_group_stats", "pg_preview", "pg_rollout_run", "pg_rollout_restore", "pg_score_preview", "pg_rollout_host_on", "pg_step_reward"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _p(t) -> Optional[int]:
    """Device (or host) address of a tensor; None -> NULL; ints pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensors passed to the library must be contiguous")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(rc: int, what: str):
    if rc != OK:
        raise PgError(rc, what)


def make_config(n_groups: int, n_expand: int, elems: int, n_steps: int,
                stages: Sequence[Sequence[int]], seed: int, vel_dtype: int, *, group_offset: int = 0,
                logp_mean: bool = False, adv_eps: float = 1e-6) -> Config:
    n = len(stages)
    steps = (ctypes.c_int32 * max(n, 1))(*[int(s) for s, _ in stages])
    keeps = (ctypes.c_int32 * max(n, 1))(*[int(k) for _, k in stages])
    cfg = Config(n_groups, n_expand, elems, n_steps, n,
                 ctypes.cast(steps, ctypes.POINTER(ctypes.c_int32)),
                 ctypes.cast(keeps, ctypes.POINTER(ctypes.c_int32)),
                 seed & 0xFFFFFFFFFFFFFFFF, group_offset, vel_dtype, 1 if logp_mean else 0, adv_eps)
    cfg._keepalive = (steps, keeps)
    return cfg


def rollout_init(cfg: Config) -> int:
    h = ctypes.c_void_p()
    _check(lib().pg_rollout_init(ctypes.byref(cfg), ctypes.byref(h)), "pg_rollout_init")
    return h.value


def rollout_destroy(h: int) -> None:
    _check(lib().pg_rollout_destroy(h), "pg_rollout_destroy")


def rollout_reset(h: int, stream=None) -> None:
    _check(lib().pg_rollout_reset(h, _stream(stream)), "pg_rollout_reset")


def rollout_restore(h: int, next_step: int, stages_done: int, traj_ids, stream=None) -> None:
    _check(lib().pg_rollout_restore(h, next_step, stages_done, _p(traj_ids), _stream(stream)),
           "pg_rollout_restore")


def rollout_status(h: int, raise_on_flags: bool = True):
    """(n_active, next_step, device_status); synchronises the device."""
    a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    rc = lib().pg_rollout_status(h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != OK and (raise_on_flags or rc not in (ENONFINITE, ETIMEOUT, EINDEX)):
        raise PgError(rc, "pg_rollout_status")
    return a.value, b.value, c.value


def step(h: int, step_index: int, coef, x_in, vel, src_rows, x_out, logp_out, stream=None) -> None:
    c = StepCoef(*coef)
    _check(lib().pg_step(h, step_index, ctypes.byref(c), _p(x_in), _p(vel), _p(src_rows), _p(x_out),
                         _p(logp_out), _stream(stream)), "pg_step")


def step_reward(h: int, step_index: int, coef, x_in, vel, src_rows, x_out, logp_out, reward_out,
                stream=None) -> None:
    """pg_step that also writes the mean of every updated latent (the final-reward stand-in)."""
    c = StepCoef(*coef)
    _check(lib().pg_step_reward(h, step_index, ctypes.byref(c), _p(x_in), _p(vel), _p(src_rows), _p(x_out),
                                _p(logp_out), _p(reward_out), _stream(stream)), "pg_step_reward")


def score(h: int, coef, x, vel, scores_out, preview_out=None, stream=None) -> None:
    c = PreviewCoef(*coef)
    _check(lib().pg_score(h, ctypes.byref(c), _p(x), _p(vel), _p(scores_out), _p(preview_out),
                          _stream(stream)), "pg_score")


def score_preview(h: int, coef, x, vel, scores_out, preview_out, stream=None) -> None:
    """Scores and the preview x_hat (fp32 or bf16 tensor, by its dtype) in one pass."""
    c = PreviewCoef(*coef)
    dt = VEL_BF16 if preview_out is not None and preview_out.dtype == torch.bfloat16 else VEL_F32
    _check(lib().pg_score_preview(h, ctypes.byref(c), _p(x), _p(vel), _p(scores_out), _p(preview_out), dt,
                                  _stream(stream)), "pg_score_preview")


def preview(h: int, coef, x, vel, out, stream=None) -> None:
    """x_hat = p_x x + p_v vel into `out` (fp32 or bf16 tensor)."""
    c = PreviewCoef(*coef)
    dt = VEL_BF16 if out.dtype == torch.bfloat16 else VEL_F32
    _check(lib().pg_preview(h, ctypes.byref(c), _p(x), _p(vel), _p(out), dt, _stream(stream)), "pg_preview")


def prune_ovf(h: int, stage: int, scores, keep_idx, src_rows=None, sel_var=None, stream=None) -> None:
    _check(lib().pg_prune_ovf(h, stage, _p(scores), _p(keep_idx), _p(src_rows), _p(sel_var),
                              _stream(stream)), "pg_prune_ovf")


def prune_uniform(h: int, stage: int, keep_idx, src_rows=None, stream=None) -> None:
    _check(lib().pg_prune_uniform(h, stage, _p(keep_idx), _p(src_rows), _stream(stream)), "pg_prune_uniform")


def group_stats(n_groups: int, n: int, scores, delta: float, mean=None, std=None, clustered_frac=None,
                stream=None) -> None:
    _check(lib().pg_group_stats(n_groups, n, _p(scores), delta, _p(mean), _p(std), _p(clustered_frac),
                                _stream(stream)), "pg_group_stats")


def compact(h: int, keep_idx, src, dst, row_bytes: int, stream=None) -> None:
    _check(lib().pg_compact(h, _p(keep_idx), _p(src), _p(dst), row_bytes, _stream(stream)),
           "pg_compact")


def advantages(h: int, rewards, adv, mean=None, std=None, stream=None) -> None:
    _check(lib().pg_advantages(h, _p(rewards), _p(adv), _p(mean), _p(std), _stream(stream)),
           "pg_advantages")


def policy_logprob(h: int, coef, x, x_next, vel, vel_ref, logp_out, kl_out=None, stream=None) -> None:
    c = StepCoef(*coef)
    _check(lib().pg_policy_logprob(h, ctypes.byref(c), _p(x), _p(x_next), _p(vel), _p(vel_ref),
                                   _p(logp_out), _p(kl_out), _stream(stream)), "pg_policy_logprob")


def policy_objective(h: int, n_steps: int, logp_new, logp_old, kl, adv, clip_eps: float, beta: float,
                     ratio, dlogp, objective, stream=None) -> None:
    _check(lib().pg_policy_objective(h, n_steps, _p(logp_new), _p(logp_old), _p(kl), _p(adv), clip_eps,
                                     beta, _p(ratio), _p(dlogp), _p(objective), _stream(stream)),
           "pg_policy_objective")


def policy_backward(h: int, coef, x, x_next, vel, vel_ref, dlogp, dkl: float, grad_vel, stream=None) -> None:
    c = StepCoef(*coef)
    _check(lib().pg_policy_backward(h, ctypes.byref(c), _p(x), _p(x_next), _p(vel), _p(vel_ref),
                                    _p(dlogp), dkl, _p(grad_vel), _stream(stream)), "pg_policy_backward")


def ovf_select_batched(n_groups: int, n: int, k: int, scores, keep_idx, kept_scores=None, adv=None,
                       adv_eps: float = 1e-6, status=None, stream=None) -> None:
    _check(lib().pg_ovf_select_batched(n_groups, n, k, _p(scores), _p(keep_idx), _p(kept_scores),
                                       _p(adv), adv_eps, _p(status), _stream(stream)),
           "pg_ovf_select_batched")


def score_static(n_rows: int, elems: int, vel_dtype: int, coef, x, vel, scores_out, stream=None) -> None:
    """pg_score without a handle and without any allocation: the reduction scratch is a fixed
    array inside the library (see pg_score_static for its limits and sharing rules)."""
    c = PreviewCoef(*coef)
    _check(lib().pg_score_static(n_rows, elems, vel_dtype, ctypes.byref(c), _p(x), _p(vel),
                                 _p(scores_out), _stream(stream)), "pg_score_static")


def survivor_rows(h: int, keep_idx_packed, rows_out, stream=None) -> None:
    """rows_out [T, G*K] int32: row of every final survivor at every step."""
    _check(lib().pg_survivor_rows(h, _p(keep_idx_packed), _p(rows_out), _stream(stream)), "pg_survivor_rows")


def survivor_logp(h: int, rows, logp_packed, logp_out, stream=None) -> None:
    """logp_out [T, G*K]: the survivors' entries of the packed per-step log-probs."""
    _check(lib().pg_survivor_logp(h, _p(rows), _p(logp_packed), _p(logp_out), _stream(stream)),
           "pg_survivor_logp")


def gather_rows(h: int, rows, n_out: int, n_in: int, src, dst, row_bytes: int, stream=None) -> None:
    _check(lib().pg_gather_rows(h, _p(rows), n_out, n_in, _p(src), _p(dst), row_bytes, _stream(stream)),
           "pg_gather_rows")


def selftest_bounded_wait(h: int, stream=None) -> None:
    """Makes the library's bounded device-side wait run out once (sets status bit 1)."""
    _check(lib().pg_selftest_bounded_wait(h, _stream(stream)), "pg_selftest_bounded_wait")


def rollout_traj_ids(h: int, dst, stream=None) -> None:
    _check(lib().pg_rollout_traj_ids(h, _p(dst), _stream(stream)), "pg_rollout_traj_ids")


def philox_raw(n: int, ctr, key, out, stream=None) -> None:
    _check(lib().pg_philox_raw(n, _p(ctr), _p(key), _p(out), _stream(stream)), "pg_philox_raw")


def normal_rows(seed: int, step_index: int, stream_id: int, n_rows: int, d: int, traj_id, out,
                stream=None) -> None:
    _check(lib().pg_normal_rows(seed & 0xFFFFFFFFFFFFFFFF, step_index, stream_id, n_rows, d,
                                _p(traj_id), _p(out), _stream(stream)), "pg_normal_rows")


def rollout_host_workspace_bytes(cfg: Config) -> int:
    return int(lib().pg_rollout_host_workspace_bytes(ctypes.byref(cfg)))


def rollout_host(cfg: Config, step_coefs, preview_coefs, x0, vel_steps, stage_scores, final_rewards,
                 x_final, logp, keep_idx, adv, traj_id, workspace) -> int:
    """Whole rollout from host tensors (see pg_rollout_host).  Returns the status code, raising
    for anything but OK / ENONFINITE."""
    sc = (StepCoef * len(step_coefs))(*[StepCoef(*c) for c in step_coefs])
    npc = max(len(preview_coefs), 1)
    pc = (PreviewCoef * npc)(*[PreviewCoef(*c) for c in preview_coefs])
    vs = (ctypes.c_void_p * len(vel_steps))(*[_p(v) for v in vel_steps])
    ss = None
    if stage_scores is not None:
        ss = (ctypes.c_void_p * max(len(stage_scores), 1))(*[_p(s) for s in stage_scores])
    rc = lib().pg_rollout_host(ctypes.byref(cfg), sc, pc, _p(x0), vs, ss, _p(final_rewards),
                               _p(x_final), _p(logp), _p(keep_idx), _p(adv), _p(traj_id),
                               _p(workspace), workspace.numel() * workspace.element_size())
    if rc not in (OK, ENONFINITE):
        raise PgError(rc, "pg_rollout_host")
    return rc


class HostArgs:
    """Marshalled arguments of pg_rollout_host_on, built once and reused call after call."""

    def __init__(self, step_coefs, preview_coefs, vel_steps, stage_scores=None):
        self.sc = (StepCoef * len(step_coefs))(*[StepCoef(*c) for c in step_coefs])
        self.pc = (PreviewCoef * max(len(preview_coefs), 1))(*[PreviewCoef(*c) for c in preview_coefs])
        self.vs = (ctypes.c_void_p * len(vel_steps))(*[_p(v) for v in vel_steps])
        self.ss = None
        if stage_scores is not None:
            self.ss = (ctypes.c_void_p * max(len(stage_scores), 1))(*[_p(s) for s in stage_scores])
        self.keep = (vel_steps, stage_scores)      # the host tensors must outlive the calls


def rollout_host_on(h: int, args: "HostArgs", x0, final_rewards, x_final, logp, keep_idx, adv, traj_id,
                    workspace) -> int:
    """Whole rollout from host tensors on an existing handle (see pg_rollout_host_on): no
    allocation per call.  Returns the status code, raising for anything but OK / ENONFINITE."""
    rc = lib().pg_rollout_host_on(h, args.sc, args.pc, _p(x0), args.vs, args.ss, _p(final_rewards),
                                  _p(x_final), _p(logp), _p(keep_idx), _p(adv), _p(traj_id),
                                  _p(workspace), workspace.numel() * workspace.element_size())
    if rc not in (OK, ENONFINITE):
        raise PgError(rc, "pg_rollout_host_on")
    return rc


def rollout_run_workspace_bytes(cfg: Config) -> int:
    return int(lib().pg_rollout_run_workspace_bytes(ctypes.byref(cfg)))


class RunArgs:
    """Marshalled arguments of pg_rollout_run, built once and reusable (e.g. under graph capture)."""

    def __init__(self, step_coefs, preview_coefs, vel_steps, stage_scores=None):
        self.sc = (StepCoef * len(step_coefs))(*[StepCoef(*c) for c in step_coefs])
        self.pc = (PreviewCoef * max(len(preview_coefs), 1))(*[PreviewCoef(*c) for c in preview_coefs])
        self.vs = (ctypes.c_void_p * len(vel_steps))(*[_p(v) for v in vel_steps])
        self.ss = None
        if stage_scores is not None:
            self.ss = (ctypes.c_void_p * max(len(stage_scores), 1))(*[_p(t) for t in stage_scores])
        self.keep = (vel_steps, stage_scores)
        self.out = RolloutOutputs()


def rollout_run(h: int, args: "RunArgs", x0, final_rewards, workspace, stream=None) -> RolloutOutputs:
    """pg_rollout_run: the whole schedule from device tensors, enqueued on one stream."""
    _check(lib().pg_rollout_run(h, args.sc, args.pc, _p(x0), args.vs, args.ss, _p(final_rewards),
                                _p(workspace), workspace.numel() * workspace.element_size(),
                                ctypes.byref(args.out), _stream(stream)), "pg_rollout_run")
    return args.out


def strerror(code: int) -> str:
    return lib().pg_strerror(code).decode()


def launch_count() -> int:
    return int(lib().pg_launch_count())
