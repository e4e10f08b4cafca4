"""Thin driver over the C ABI: owns the device buffers of one rollout batch and issues the
library calls in schedule order.  Allocation and streams are torch's; every number is computed
by the library's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import torch

from . import binding as B


@dataclass
class RolloutOutput:
    x_final: torch.Tensor                 # [G*K, d] fp32
    logp: List[torch.Tensor]              # per step [rows taking that step] fp32
    traj_id: torch.Tensor                 # [G*K] int32
    stage_scores: List[torch.Tensor] = field(default_factory=list)
    stage_keep: List[torch.Tensor] = field(default_factory=list)
    stage_var: List[torch.Tensor] = field(default_factory=list)
    rewards: Optional[torch.Tensor] = None
    adv: Optional[torch.Tensor] = None
    mean: Optional[torch.Tensor] = None
    std: Optional[torch.Tensor] = None


def initial_latents(seed: int, n_groups: int, n_expand: int, elems: int, group_offset: int = 0,
                    device=None) -> torch.Tensor:
    """x_0 ~ N(0, I) for G * N0 trajectories from the library's counter-based generator (noise
    stream 1, keyed by the global trajectory id), so any sharding of the groups draws the same
    latents.  fp32 [G * N0, d]."""
    dev = device or torch.device("cuda", torch.cuda.current_device())
    rows = n_groups * n_expand
    ids = torch.arange(group_offset * n_expand, group_offset * n_expand + rows, device=dev, dtype=torch.int32)
    out = torch.empty(rows, elems, device=dev, dtype=torch.float32)
    B.normal_rows(seed, 0, 1, rows, elems, ids, out)
    return out


class Rollout:
    """One Expand-and-Prune batch on the current CUDA device."""

    def __init__(self, n_groups: int, n_expand: int, elems: int, n_steps: int,
                 stages: Sequence[Tuple[int, int]], seed: int, vel_dtype: torch.dtype,
                 adv_eps: float = 1e-6, group_offset: int = 0, logp_mean: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("the rollout library needs a CUDA device; there is no CPU path")
        self.G, self.N0, self.d, self.T = n_groups, n_expand, elems, n_steps
        self.stages = [(int(s), int(k)) for s, k in stages]
        self.vel_dtype = vel_dtype
        vd = B.VEL_BF16 if vel_dtype == torch.bfloat16 else B.VEL_F32
        self.cfg = B.make_config(n_groups, n_expand, elems, n_steps, self.stages, seed, vd,
                                 group_offset=group_offset, logp_mean=logp_mean, adv_eps=adv_eps)
        self.h = B.rollout_init(self.cfg)
        dev = torch.device("cuda", torch.cuda.current_device())
        rows = n_groups * n_expand
        self.dev = dev
        self.x = [torch.empty(rows, elems, device=dev, dtype=torch.float32) for _ in range(2)]
        self.cur = 0
        self.k_cur = n_expand
        self.trace = None
        self.scores = torch.empty(rows, device=dev, dtype=torch.float32)
        self.src_rows = torch.empty(rows, device=dev, dtype=torch.int32)
        self.rewards = torch.empty(rows, device=dev, dtype=torch.float32)
        total = 0
        k = n_expand
        st = dict(self.stages)
        self.rows_at = []
        for s in range(n_steps):
            k = st.get(s, k)
            self.rows_at.append(n_groups * k)
            total += n_groups * k
        self.logp_all = torch.empty(total, device=dev, dtype=torch.float32)
        self.keep = [torch.empty(n_groups * k, device=dev, dtype=torch.int32) for _, k in self.stages]
        self.sel_var = [torch.empty(n_groups, device=dev, dtype=torch.float32) for _ in self.stages]
        self.adv = torch.empty(n_groups * (self.stages[-1][1] if self.stages else n_expand),
                               device=dev, dtype=torch.float32)
        self.mean = torch.empty(n_groups, device=dev, dtype=torch.float32)
        self.std = torch.empty(n_groups, device=dev, dtype=torch.float32)

    def close(self):
        if getattr(self, "h", None):
            torch.cuda.synchronize()
            B.rollout_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def n_active(self) -> int:
        return self.G * self.k_cur

    def reset(self):
        B.rollout_reset(self.h)
        self.cur = 0
        self.k_cur = self.N0

    def _timed(self, kind: str, rows: int, fn):
        """Runs one library call, bracketed by CUDA events when tracing is on."""
        if self.trace is None:
            fn()
            return
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        self.trace.append((kind, rows, a, b))

    def run(self, x0: torch.Tensor,
            step_coef: Callable[[int], Tuple[float, float, float]],
            preview_coef: Callable[[int], Tuple[float, float]],
            velocity: Callable[[int, torch.Tensor], torch.Tensor],
            external_scores: Optional[Callable[[int], torch.Tensor]] = None,
            final_rewards: Optional[Callable[[], torch.Tensor]] = None,
            record_scores: bool = False, trace: Optional[list] = None,
            selector: str = "ovf") -> RolloutOutput:
        """Runs the whole schedule.  ``velocity(step, x_active)`` returns the prediction for the
        currently active rows; ``external_scores(stage)`` / ``final_rewards()`` return device
        fp32 tensors when the scores come from outside (else the preview mean / latent mean).
        x0 is only read (step 0 writes into the driver's own buffer).  With ``trace`` (a list),
        every library call is bracketed by CUDA events: (kind, rows, start, end) is appended.
        ``selector`` is "ovf" (Optimal Variance Filtering) or "uniform" (the random-subset
        baseline; scores are then neither computed nor needed)."""
        if selector not in ("ovf", "uniform"):
            raise ValueError("selector must be 'ovf' or 'uniform'")
        self.reset()
        self.trace = trace
        out = RolloutOutput(x_final=None, logp=[], traj_id=None)
        stage_i, off = 0, 0
        x_cur = x0                      # current latent tensor (x0 first, then own buffers)
        for s in range(self.T):
            vel = velocity(s, x_cur[: self.n_active])
            src = None
            if stage_i < len(self.stages) and self.stages[stage_i][0] == s and selector == "uniform":
                self._timed("prune", self.n_active, lambda: B.prune_uniform(
                    self.h, stage_i, self.keep[stage_i], self.src_rows))
                self.k_cur = self.stages[stage_i][1]
                src = self.src_rows
                stage_i += 1
            elif stage_i < len(self.stages) and self.stages[stage_i][0] == s:
                if external_scores is not None:
                    sc = external_scores(stage_i)
                else:
                    sc = self.scores[: self.n_active]
                    self._timed("score", self.n_active, lambda: B.score(
                        self.h, preview_coef(s), x_cur, vel, sc))
                if record_scores:
                    out.stage_scores.append(sc.clone())
                self._timed("prune", self.n_active, lambda: B.prune_ovf(
                    self.h, stage_i, sc, self.keep[stage_i], self.src_rows, self.sel_var[stage_i]))
                self.k_cur = self.stages[stage_i][1]
                src = self.src_rows
                stage_i += 1
            rows = self.n_active
            lp = self.logp_all[off: off + rows]
            if src is not None or x_cur is x0:
                dst = self.x[self.cur ^ 1] if x_cur is self.x[self.cur] else self.x[self.cur]
            else:
                dst = x_cur                                 # in place
            if s == self.T - 1 and final_rewards is None:
                # the last step also reduces the stand-in reward (mean of x_T) from its registers
                rw_fused = self.rewards[:rows]
                self._timed("step", rows, lambda: B.step_reward(self.h, s, step_coef(s), x_cur, vel, src, dst,
                                                                lp, rw_fused))
            else:
                self._timed("step", rows, lambda: B.step(self.h, s, step_coef(s), x_cur, vel, src, dst, lp))
            if dst is not x_cur:
                if x_cur is not x0:
                    self.cur ^= 1
                x_cur = dst
            out.logp.append(lp)
            off += rows
        rows = self.n_active
        if final_rewards is not None:
            rw = final_rewards()
        else:
            rw = self.rewards[:rows]                      # written by the last step
        self._timed("advantages", rows, lambda: B.advantages(self.h, rw, self.adv, self.mean, self.std))
        ids = torch.empty(rows, device=self.dev, dtype=torch.int32)
        B.rollout_traj_ids(self.h, ids)
        out.x_final = x_cur[:rows]
        out.traj_id = ids
        self.trace = None
        out.stage_keep = list(self.keep)
        out.stage_var = list(self.sel_var)
        out.rewards, out.adv, out.mean, out.std = rw, self.adv, self.mean, self.std
        return out


class NativeRollout:
    """Whole rollouts through pg_rollout_run: one library call enqueues every launch of the
    schedule on the current stream (device-resident inputs), optionally replayed as a CUDA graph
    when the rollout is launch-bound."""

    def __init__(self, ro: Rollout, step_coefs, preview_coefs, vel_steps, stage_scores=None):
        self.ro = ro
        self.args = B.RunArgs(step_coefs, preview_coefs, vel_steps, stage_scores)
        self.ws = torch.empty(B.rollout_run_workspace_bytes(ro.cfg), dtype=torch.uint8, device=ro.dev)
        self.graph = None
        self.x0 = None

    def _view(self, ptr: int, count: int, dtype: torch.dtype) -> torch.Tensor:
        off = ptr - self.ws.data_ptr()
        size = torch.empty(0, dtype=dtype).element_size()
        return self.ws[off: off + count * size].view(dtype)

    def run(self, x0: torch.Tensor, final_rewards: Optional[torch.Tensor] = None) -> RolloutOutput:
        o = B.rollout_run(self.ro.h, self.args, x0, final_rewards, self.ws)
        return self._outputs(o)

    def capture(self, x0: torch.Tensor, final_rewards: Optional[torch.Tensor] = None) -> None:
        """Records one rollout from x0 into a CUDA graph; replay() then re-runs it."""
        self.x0 = x0
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            B.rollout_run(self.ro.h, self.args, x0, final_rewards, self.ws)      # warm-up, loads kernels
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.out_struct = B.rollout_run(self.ro.h, self.args, x0, final_rewards, self.ws)

    def replay(self) -> RolloutOutput:
        self.graph.replay()
        return self._outputs(self.out_struct)

    def _outputs(self, o) -> RolloutOutput:
        ro = self.ro
        n, d = int(o.n_final), ro.d
        logp_all = self._view(o.logp, int(o.n_logp), torch.float32)
        keep_all = self._view(o.keep_idx, int(o.n_keep), torch.int32) if o.n_keep else None
        out = RolloutOutput(x_final=self._view(o.x_final, n * d, torch.float32).view(n, d), logp=[],
                            traj_id=self._view(o.traj_id, n, torch.int32))
        off = 0
        for rows in ro.rows_at:
            out.logp.append(logp_all[off: off + rows])
            off += rows
        off = 0
        for _, k in ro.stages:
            out.stage_keep.append(keep_all[off: off + ro.G * k])
            off += ro.G * k
        out.adv = self._view(o.adv, n, torch.float32)
        ws_lo, ws_hi = self.ws.data_ptr(), self.ws.data_ptr() + self.ws.numel()
        if ws_lo <= o.rewards < ws_hi:
            out.rewards = self._view(o.rewards, n, torch.float32)
        return out


class GraphedRollout:
    """The step-by-step driver recorded once into a CUDA graph and replayed, network included.

    For launch-bound rollouts whose predictions depend on the current latents (a denoiser, or a
    stand-in such as an affine field, written as capturable torch ops): ``velocity(step, x)`` and
    the optional score / reward callbacks are traced during capture, so a replay re-runs the
    library's kernels and the network's kernels from x0's current contents without any Python in
    between.  The callbacks must not synchronise or move data to the host."""

    def __init__(self, ro: Rollout, x0: torch.Tensor, step_coef, preview_coef, velocity,
                 external_scores=None, final_rewards=None):
        self.ro, self.x0 = ro, x0
        run = lambda: ro.run(x0, step_coef, preview_coef, velocity, external_scores=external_scores,
                             final_rewards=final_rewards)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            run()                                   # warm-up outside the capture (loads kernels)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.out = run()

    def replay(self) -> RolloutOutput:
        self.graph.replay()
        return self.out

