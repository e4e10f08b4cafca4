#!/usr/bin/env python
"""Benchmark of the Expand-and-Prune rollout hot path.

One "step" of this benchmark is one whole rollout of the large workload (64 prompt groups,
64 -> 32 -> 16 (-> 16) trajectories pruned at steps 2, 5, 8 of 28, 16x128x128 fp32 latents, bf16
predictions): SDE step + log-prob at every step, latent scoring + OVF + (folded) compaction at
every stage, group advantages at the end.  The reported value is latent-steps per second
(one latent-step = one trajectory advanced by one SDE step, log-prob included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs its own 64
groups (weak scaling, groups are independent, no data-path collective); times are taken on the
device and the maximum over ranks is used.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

STEP_PROFILE = os.path.join(ROOT, "profiles", "step_kernel_bf16_256rows.txt")
STEP_SOURCES = [os.path.join(ROOT, "paper_2512_15347_b200", "csrc", f) for f in ("pg_step.cu", "pg_common.cuh")]


def _sources_sha256(paths=STEP_SOURCES):
    import hashlib
    h = hashlib.sha256()
    for p in paths:
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def step_traffic_ratio(profile=STEP_PROFILE):
    """DRAM bytes over algorithmic bytes of the step kernel, read from the committed ncu summary:
    its `dram__bytes_read.sum` / `dram__bytes_write.sum` lines (first captured launch) and its
    `algorithmic_bytes` line.  The summary also records the SHA-256 of the kernel's sources at
    capture time; when the sources have changed since, the counters no longer describe the kernel
    and None is returned (the bench line then carries "traffic": null)."""
    import re
    try:
        text = open(profile).read()
    except OSError:
        return None, "no ncu summary"
    sha = re.search(r"source_sha256:\s*([0-9a-f]{64})", text)
    if not sha or sha.group(1) != _sources_sha256():
        return None, "kernel sources changed since the ncu capture"
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    vals = {}
    for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(re.escape(key) + r"\s+([0-9.eE+-]+)\s*(byte|Kbyte|Mbyte|Gbyte)", text)
        if not m:
            return None, "ncu summary lacks " + key
        vals[key] = float(m.group(1)) * unit[m.group(2)]
    alg = re.search(r"algorithmic_bytes:\s*([0-9]+)", text)
    if not alg:
        return None, "ncu summary lacks algorithmic_bytes"
    return sum(vals.values()) / float(alg.group(1)), os.path.relpath(profile, ROOT)


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.lower().startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    import platform
    return platform.processor() or platform.machine()


# the headline metric has three components: `value` is the first (latent-steps/s), the achieved HBM
# GB/s is in `roofline` / `hbm_gbs_whole_rollout` / `prune_stage_gbs`, OVF groups/s in `ovf_microbench`
METRIC = "latent-steps/s & achieved HBM GB/s (SDE step+logprob+OVF prune); OVF groups/s"
UNIT = "latent-steps/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        rows = [r for r in self.rows if t0 - 0.05 <= r[0] <= t1 + 0.15] or self.rows
        for _, line in rows:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                  "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ CPU oracle timing

class OracleSample:
    """A bounded sample of the workload for the CPU oracle: the first `groups` prompt groups with
    the full schedule and full-length latents (groups are independent, cost is linear in groups)."""

    def __init__(self, w, groups: int):
        from paper_2512_15347_b200 import workloads as wl
        import torch
        self.w = w
        self.sw = sw = wl.scaled(w, n_groups=groups)
        self.x0 = wl.initial_latents(sw).numpy()
        if w.velocity == "affine":
            a, b = wl.affine_field(sw)
            self.velocity = lambda s, x, traj: wl.affine_velocity(torch.from_numpy(x), a, b).numpy()
        elif w.velocity == "eps":
            zs = [wl.normal_noise(sw, s, groups * w.rows_before(s)) for s in range(w.n_steps)]
            self.velocity = lambda s, x, traj: wl.as_numpy_velocity(
                wl.eps_velocity(torch.from_numpy(x), zs[s], *wl.eps_mix(sw, s), sw.vel_dtype))
        else:
            vels = [wl.as_numpy_velocity(wl.normal_velocity(sw, s, groups * w.rows_before(s)))
                    for s in range(w.n_steps)]
            self.velocity = lambda s, x, traj: vels[s]
        self.ext = self.fin = None
        if w.scores == "external":
            self.ext = lambda stage, traj: wl.sd3_stage_scores(sw, stage, traj)
            self.fin = lambda x, traj: wl.sd3_stage_scores(sw, 99, traj)
        self.desc = (f"first {groups} of {w.n_groups} prompt groups, full schedule, full-length latents "
                     f"({self.sw.traj_steps} of {w.traj_steps} latent-steps)")

    def run(self) -> float:
        """One oracle rollout of the sample; returns seconds."""
        import oracle
        sw = self.sw
        t0 = time.perf_counter()
        oracle.rollout(self.x0, sw.n_groups, sw.n_expand, sw.n_steps, sw.stages, sw.seed, sw.step_coef,
                       sw.preview_coef, self.velocity, external_scores=self.ext, final_rewards=self.fin,
                       adv_eps=sw.adv_eps)
        return time.perf_counter() - t0


ORACLE_GROUPS = 8
# smaller workloads reported beside the bench line: (name, prompt groups of the oracle's sample)
OTHER_WORKLOADS = (('sd3', 4), ('sd15', 8), ('tiny', 1))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2512_15347_b200 import workloads as wl
    w = wl.load_workload(args.config) if args.config else wl.WORKLOADS[args.workload]
    small = OracleSample(w, 1)
    t1 = min([small.run() for _ in range(max(args.warmup, 1))])
    # bounded sample: as many groups (up to ORACLE_GROUPS) as keep the timed steps near two minutes
    groups = max(1, min(ORACLE_GROUPS, w.n_groups, int(120.0 / (max(args.steps, 1) * t1))))
    sample = small if groups == 1 else OracleSample(w, groups)
    times = [sample.run() for _ in range(args.steps)]
    mean_sec = sum(times) / len(times)
    value = sample.sw.traj_steps / mean_sec
    threads = oracle.num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": _config(w, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "cpu_model": cpu_model(),
                             "kind": "oracle", "sample": sample.desc + "; warm-up on 1 group"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def _config(w, args):
    return {"workload": f"{w.name}: {w.n_groups} groups x {w.n_expand} -> "
                        + " -> ".join(str(k) for _, k in w.stages)
                        + f" at steps {[s for s, _ in w.stages]} of {w.n_steps}, d={w.elems}, "
                        f"fp32 latents, {w.vel_dtype} predictions, seed {w.seed}",
            "groups_per_gpu": w.n_groups, "latent_steps_per_rollout": w.traj_steps,
            "l2": ("inputs larger than L2: no flush" if w.n_groups * w.n_expand * w.elems * 4 > 256e6
                   else "state fits L2 (L2-assisted numbers, launch-bound workload)")
                  + " (state %.3f GB, predictions %.3f GB per rollout)"
                  % (w.n_groups * w.n_expand * w.elems * 4 / 1e9,
                     w.element_steps * (2 if w.vel_dtype == "bf16" else 4) / 1e9),
            "parallelism": f"groups sharded over {args.gpus} GPU(s), no collective"}


# ------------------------------------------------------------------ GPU arm

def _gpu_inputs(w, wr, ro, dev, rank):
    """Seeded device inputs of one workload: initial latents, the per-step predictions (or the
    stand-in network for the affine field), and the stand-in reward model of the workloads whose
    scores come from outside."""
    import torch
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200 import workloads as wl
    from paper_2512_15347_b200 import sharding
    x0 = wl.initial_latents(wr, device=dev)
    ext = fin = vels = None
    if w.velocity == "affine":
        a_c, b_c = wl.affine_field(wr, device=dev)
        velocity = lambda s, x: wl.affine_velocity(x, a_c, b_c)   # stand-in network, inside the timing
    elif w.velocity == "eps":
        zs = [wl.normal_noise(wr, s, w.n_groups * w.rows_before(s), device=dev) for s in range(w.n_steps)]
        mix = [wl.eps_mix(wr, s) for s in range(w.n_steps)]
        # stand-in noise-prediction network (3 torch ops per step), inside the timing
        velocity = lambda s, x: wl.eps_velocity(x, zs[s], *mix[s], wr.vel_dtype)
    else:
        vels = [wl.normal_velocity(wr, s, w.n_groups * w.rows_before(s), device=dev)
                for s in range(w.n_steps)]
        velocity = lambda s, x: vels[s]
    if w.scores == "external":
        # stand-in reward model: one score table per stage, looked up by original trajectory
        tables = [torch.from_numpy(wl.clustered_scores(w.n_groups, w.n_expand, wr.seed, st, cluster_sigma=0.05,
                                                       outlier_frac=0.15, outlier_scale=0.3, nu=3.0)
                                   ).reshape(-1).to(dev) for st in list(range(len(w.stages))) + [99]]
        base = sharding.weak_shard(w.n_groups, rank)[0] * w.n_expand

        def lookup(table):
            ids = torch.empty(ro.n_active, device=dev, dtype=torch.int32)
            B.rollout_traj_ids(ro.h, ids)
            return table[(ids - base).long()]
        ext = lambda stage: lookup(tables[stage])
        fin = lambda: lookup(tables[-1])
    return x0, velocity, ext, fin, vels


def _other_workload(name, dev, reps, peak):
    """One of the smaller workloads through the same step-by-step driver: ms per rollout,
    latent-steps/s and the step kernel's algorithmic GB/s (CUDA events around every call)."""
    import torch
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200 import workloads as wl
    from paper_2512_15347_b200.rollout import Rollout
    w = wl.WORKLOADS[name]
    dt = torch.bfloat16 if w.vel_dtype == "bf16" else torch.float32
    ro = Rollout(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, dt, adv_eps=w.adv_eps)
    x0, velocity, ext, fin, vels = _gpu_inputs(w, w, ro, dev, 0)
    run = lambda trace=None: ro.run(x0, w.step_coef, w.preview_coef, velocity, external_scores=ext,
                                    final_rewards=fin, trace=trace)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    traces = []
    a.record()
    for _ in range(reps):
        tr = []
        run(trace=tr)
        traces.append(tr)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    step_ms = sum(e0.elapsed_time(e1) for tr in traces for kind, _, e0, e1 in tr if kind == "step") / reps
    step_gbs = w.traj_steps * (w.elems * (8 + (2 if w.vel_dtype == "bf16" else 4)) + 4) / (step_ms * 1e-3) / 1e9
    state_mb = w.n_groups * w.n_expand * w.elems * 4 / 1e6
    graph = None
    if w.velocity == "normal" and w.scores == "preview":
        # the whole rollout as one library call, captured once in a CUDA graph and replayed
        from paper_2512_15347_b200.rollout import NativeRollout
        nat = NativeRollout(ro, [w.step_coef(s) for s in range(w.n_steps)],
                            [w.preview_coef(s) for s, _ in w.stages], vels)
        nat.capture(x0)
        nat.graph.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            nat.graph.replay()
        b.record()
        torch.cuda.synchronize()
        gms = a.elapsed_time(b) / reps
        graph = {"ms_per_rollout": gms, "latent_steps_per_s": w.traj_steps / (gms * 1e-3)}
        del nat
    elif w.velocity in ("affine", "eps") and w.scores == "preview":
        # predictions depend on the latents: the step-by-step driver with the stand-in network's
        # torch ops recorded into one CUDA graph
        from paper_2512_15347_b200.rollout import GraphedRollout
        gr = GraphedRollout(ro, x0, w.step_coef, w.preview_coef, velocity)
        gr.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            gr.replay()
        b.record()
        torch.cuda.synchronize()
        gms = a.elapsed_time(b) / reps
        graph = {"ms_per_rollout": gms, "latent_steps_per_s": w.traj_steps / (gms * 1e-3),
                 "note": "stand-in network (a few torch ops per step) inside the graph"}
        del gr
    ro.close()
    e2e_small = None
    if w.velocity == "normal" and w.scores == "preview":
        import argparse
        e = run_e2e(B, wl, w, w, 0, None, dev, argparse.Namespace(steps=max(reps, 10)))
        e2e_small = {"per_call_handle_ms": e["ms_per_step"], "existing_handle_ms": e["on_existing_handle"]["ms_per_step"],
                     "existing_handle_latent_steps_per_s": e["on_existing_handle"]["value"],
                     "note": "host buffers in and out; pg_rollout_host (handle per call) vs pg_rollout_host_on"}
    return {"ms_per_rollout": ms, "e2e_host": e2e_small, "cuda_graph_replay": graph, "latent_steps_per_s": w.traj_steps / (ms * 1e-3), "step_gbs": step_gbs,
            "step_frac_of_peak": step_gbs / peak,
            "regime": ("HBM-streaming" if state_mb > 256 else
                       f"state {state_mb:.1f} MB fits L2: launch-bound, GB/s is L2-assisted")}



LAUNCH_ROWS = (192, 384, 768, 1024, 2048, 4096)


def launch_size_table(B, x_a, x_b, vel, elems, peak, rows_list=LAUNCH_ROWS, reps=24,
                      step_coef=(1.0, 0.04, 0.13)):
    """Step and score launches of the streaming shape (d = `elems`, bf16 predictions) by row count:
    device time per launch and algorithmic GB/s, measured two ways - `stream`: `reps` launches
    enqueued back to back between one pair of CUDA events (how a rollout issues them; successive
    launches use different rows of the buffers, so nothing is served from L2), and `isolated`: the
    median of single launches, each between its own pair of events on an idle GPU.  x_a, x_b:
    fp32 [>= max rows, d] (read / written), vel bf16 [>= max rows, d]."""
    import torch
    out = {"elems": elems, "reps": reps, "bytes_per_element": {"step": 10, "score": 6}, "rows": {}}
    cap = min(x_a.shape[0], vel.shape[0])
    lp = torch.empty(cap, device=x_a.device)
    sc = torch.empty(cap, device=x_a.device)
    for rows in rows_list:
        if rows > cap:
            continue
        h = B.rollout_init(B.make_config(rows, 1, elems, 1 << 30, [], 3, B.VEL_BF16))
        nxt = [0]
        span = cap - rows + 1

        def step(i):
            o = (i * rows) % span
            B.step(h, nxt[0], step_coef, x_a[o:o + rows], vel[o:o + rows], None, x_b[o:o + rows], lp)
            nxt[0] += 1

        def score(i):
            o = (i * rows) % span
            B.score(h, (1.0, 0.5), x_a[o:o + rows], vel[o:o + rows], sc)

        entry = {}
        for name, fn, bpe in (("step", step, 10), ("score", score, 6)):
            for i in range(3):
                fn(i)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(reps):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            stream_us = a.elapsed_time(b) / reps * 1e3
            singles = []
            for i in range(reps):
                a.record()
                fn(i)
                b.record()
                torch.cuda.synchronize()
                singles.append(a.elapsed_time(b) * 1e3)
            singles.sort()
            iso_us = singles[len(singles) // 2]
            nbytes = rows * (elems * bpe + 4)
            entry[name] = {"stream_us": stream_us, "stream_gbs": nbytes / stream_us / 1e3,
                           "stream_frac": nbytes / stream_us / 1e3 / peak,
                           "isolated_us": iso_us, "isolated_gbs": nbytes / iso_us / 1e3}
        out["rows"][str(rows)] = entry
        torch.cuda.synchronize()
        B.rollout_destroy(h)
    return out


def run_ours(args):
    import torch
    from paper_2512_15347_b200 import binding as B
    from paper_2512_15347_b200 import workloads as wl
    from paper_2512_15347_b200 import sharding
    from paper_2512_15347_b200.rollout import Rollout

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w = wl.load_workload(args.config) if args.config else wl.WORKLOADS[args.workload]
    if args.groups:
        w = wl.scaled(w, n_groups=args.groups, name=f"{w.name}[{args.groups} groups]")

    cpu_base, cpu_others = None, {}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # before the first CUDA call: the oracle's OpenMP team is created in a clean process
        import oracle
        sample = OracleSample(w, min(ORACLE_GROUPS, w.n_groups))
        sec = min(sample.run() for _ in range(2))
        cpu_base = {"value": sample.sw.traj_steps / sec, "unit": UNIT, "cores": oracle.num_threads(),
                    "cpu_model": cpu_model(), "kind": "oracle", "sample": sample.desc + f"; best of 2 runs, {sec:.1f} s each"}
        del sample
        if w.name == "large" and not args.groups and not args.no_others:
            for name, groups in OTHER_WORKLOADS:
                ow = wl.WORKLOADS[name]
                sm = OracleSample(ow, min(groups, ow.n_groups))
                sec = min(sm.run() for _ in range(2))
                cpu_others[name] = {"value": sm.sw.traj_steps / sec, "sample": sm.desc}
                del sm

    torch.cuda.set_device(local)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:      # launched by torch.distributed.run
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        from paper_2512_15347_b200 import build as pg_build
        pg_build.build()                 # no-op when libprogrpo.so is up to date; raises if nvcc fails
    if dist is not None:
        dist.barrier()
    B.lib()
    dev = torch.device("cuda", local)
    from dataclasses import replace
    wr = replace(w, seed=w.seed + 1000 * rank)

    dt = torch.bfloat16 if w.vel_dtype == "bf16" else torch.float32
    # weak scaling: world x n_groups groups dealt out in contiguous blocks, this rank's block
    # starting at group rank * n_groups (its handle gets that offset, so trajectory ids are global)
    from paper_2512_15347_b200.sharded import ShardedRollout
    sr = ShardedRollout(world * w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, dt,
                        adv_eps=w.adv_eps, dist=dist)
    assert (sr.first, sr.count) == sharding.weak_shard(w.n_groups, rank)
    ro = sr.local
    x0, velocity, ext, fin, vels = _gpu_inputs(w, wr, ro, dev, rank)
    torch.cuda.synchronize()

    def one_rollout(trace=None):
        return ro.run(x0, w.step_coef, w.preview_coef, velocity, external_scores=ext,
                      final_rewards=fin, trace=trace)

    for _ in range(max(args.warmup, 3)):
        one_rollout()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    traces = []
    launches0 = B.launch_count()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        tr = []
        last_out = one_rollout(trace=tr)
        traces.append(tr)
    ev1.record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    launches = B.launch_count() - launches0
    clocks = sampler.stop(t_wall0, t_wall1)
    total_ms = ev0.elapsed_time(ev1)
    gathered = None
    if dist is not None:
        dist.barrier()
        total_ms = sr.max_over_ranks(total_ms, dev)
        # outside the timed region: the per-group results of all ranks in global group order
        res = sr.gather(last_out, device=dev)
        gathered = {"groups": int(res.mean.numel()), "survivors": int(res.traj_id.numel()),
                    "shards": res.shards,
                    "adv_abs_group_mean_max": float(res.adv.view(res.mean.numel(), -1).mean(dim=1).abs().max())}

    # per-kernel device times from the events recorded inside the timed region
    kinds = {}
    for tr in traces:
        for kind, rows, a, b in tr:
            d = kinds.setdefault(kind, {"ms": 0.0, "rows": 0, "launches": 0})
            d["ms"] += a.elapsed_time(b)
            d["rows"] += rows
            d["launches"] += 1
    vel_bytes = 2 if w.vel_dtype == "bf16" else 4
    step_bytes = kinds["step"]["rows"] * (w.elems * (8 + vel_bytes) + 4)
    step_gbs = step_bytes / (kinds["step"]["ms"] * 1e-3) / 1e9
    score_gbs, score_bytes = None, 0
    if "score" in kinds:
        score_bytes = kinds["score"]["rows"] * (w.elems * (4 + vel_bytes) + 4)
        score_gbs = score_bytes / (kinds["score"]["ms"] * 1e-3) / 1e9
    prune_stage_gbs = None
    if "score" in kinds and "prune" in kinds:
        ms = kinds["score"]["ms"] + kinds["prune"]["ms"]
        prune_stage_gbs = (score_bytes + kinds["prune"]["rows"] * 8) / (ms * 1e-3) / 1e9
    peak, peak_kind = _peaks()
    traffic_ratio, traffic_note = step_traffic_ratio()
    # the other half of the target: the prune stage (latent scoring + OVF selection) as one unit
    also = []
    if score_gbs is not None:
        also.append({"kernel": "score_kernel (latent score, read-only)", "bound": "hbm", "achieved": score_gbs,
                     "peak": peak, "unit": "GB/s", "frac": score_gbs / peak, "bytes_per_element": 4 + vel_bytes})
    if prune_stage_gbs is not None:
        also.append({"kernel": "score + ovf (prune stage: scoring pass and selection launch together)",
                     "bound": "hbm", "achieved": prune_stage_gbs, "peak": peak, "unit": "GB/s",
                     "frac": prune_stage_gbs / peak,
                     "bytes": "6 B per scored element + 8 B per score / kept index"})

    # OVF selection microbenchmark (4096 groups x 256 scores -> 32) on rank 0
    ovf = None
    if rank == 0:
        m = wl.OVF_MICRO
        sc = torch.from_numpy(wl.ovf_micro_scores()).to(dev)
        keep = torch.empty(m["n_groups"] * m["k"], dtype=torch.int32, device=dev)
        kept = torch.empty(m["n_groups"] * m["k"], device=dev)
        adv = torch.empty(m["n_groups"] * m["k"], device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        best = []
        for i in range(13):
            flush.zero_()                       # evict the scores from L2 between repetitions
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            B.ovf_select_batched(m["n_groups"], m["n"], m["k"], sc, keep, kept, adv, 1e-6)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                best.append(a.elapsed_time(b))
        best.sort()
        med = best[len(best) // 2]
        ovf = {"groups_per_s": m["n_groups"] / (med * 1e-3), "us_per_launch": med * 1e3,
               "workload": f"{m['n_groups']} groups x {m['n']} scores -> {m['k']} (select + index/score "
                           "compaction + advantages), L2 flushed between repetitions"}

    # the same rollout through the one-call native driver and as a replayed CUDA graph
    drivers = None
    if rank == 0 and w.velocity == "normal" and w.scores == "preview":
        from paper_2512_15347_b200.rollout import NativeRollout
        nat = NativeRollout(ro, [w.step_coef(s) for s in range(w.n_steps)],
                            [w.preview_coef(s) for s, _ in w.stages], vels)

        def time_calls(fn, reps):
            fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps
        reps = max(5, min(args.steps, 50))
        native_ms = time_calls(lambda: nat.run(x0), reps)
        nat.capture(x0)
        graph_ms = time_calls(lambda: nat.graph.replay(), reps)
        drivers = {"stepwise_ms_per_rollout": total_ms / args.steps, "native_ms_per_rollout": native_ms,
                   "graph_ms_per_rollout": graph_ms,
                   "graph_latent_steps_per_s": w.traj_steps / (graph_ms * 1e-3),
                   "note": "stepwise = one library call per kernel from Python (the timed `value`); native = "
                           "pg_rollout_run, one call per rollout; graph = that call captured and replayed"}
        del nat

    def timed(fn, reps=10):
        """Median device time (ms) of one call, after three warm-up calls."""
        ts = []
        for i in range(reps + 3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        ts.sort()
        return ts[len(ts) // 2]

    # policy-update kernels on the survivors' shape (secondary numbers; not part of `value`)
    policy = None
    if rank == 0 and w.vel_dtype == "bf16" and w.velocity == "normal":
        rows = w.n_groups * w.final_keep
        xa, xb = ro.x[0][:rows], ro.x[1][:rows]
        va, vb = vels[-1][:rows], vels[-2][:rows]
        lp = torch.empty(rows, device=dev)
        klv = torch.empty(rows, device=dev)
        dl = torch.full((rows,), 1e-3, device=dev)
        grad = torch.empty(rows, w.elems, device=dev, dtype=torch.bfloat16)
        coef = w.step_coef(0)

        t_lp = timed(lambda: B.policy_logprob(ro.h, coef, xa, xb, va, vb, lp, klv))
        t_bw = timed(lambda: B.policy_backward(ro.h, coef, xa, xb, va, vb, dl, -1e-6, grad))
        policy = {"rows": rows, "logprob_kl_gbs": rows * w.elems * 12 / (t_lp * 1e-3) / 1e9,
                  "backward_gbs": rows * w.elems * 14 / (t_bw * 1e-3) / 1e9,
                  "bytes_per_element": {"logprob_kl": 12, "backward": 14},
                  "note": "per-step kernels of the update on the survivors (x, x_next fp32; new and "
                          "reference predictions bf16; bf16 gradient), inputs larger than L2"}

    # physical compaction and preview emission on the first stage's shape (secondary numbers: the
    # rollout folds the compaction into the next step's gather and scores without emitting)
    other = None
    if rank == 0 and w.vel_dtype == "bf16" and w.velocity == "normal" and w.stages:
        k0 = w.stages[0][1]
        rows_in, rows_out = w.n_groups * w.n_expand, w.n_groups * k0
        hc = B.rollout_init(B.make_config(w.n_groups, w.n_expand, w.elems, 1, [(0, k0)], w.seed, B.VEL_BF16))
        sc0 = torch.randn(rows_in, device=dev)
        keep0 = torch.empty(rows_out, dtype=torch.int32, device=dev)
        B.prune_ovf(hc, 0, sc0, keep0)
        src_x, dst_x = ro.x[0][:rows_in], ro.x[1][:rows_out]
        t_c = timed(lambda: B.compact(hc, keep0, src_x, dst_x, w.elems * 4))
        B.rollout_destroy(hc)
        hp = B.rollout_init(B.make_config(w.n_groups, k0, w.elems, 1, [], w.seed, B.VEL_BF16))
        xs, vs = ro.x[0][:rows_out], vels[0][:rows_out]
        out16 = torch.empty(rows_out, w.elems, device=dev, dtype=torch.bfloat16)
        t_p16 = timed(lambda: B.preview(hp, (1.0, 0.5), xs, vs, out16))
        # scores and the bf16 preview in one pass (what a decoder + reward model between preview and
        # selection need), against scoring alone and against the two separate passes
        sc_out = torch.empty(rows_out, device=dev)
        t_sp16 = timed(lambda: B.score_preview(hp, (1.0, 0.5), xs, vs, sc_out, out16))
        t_s = timed(lambda: B.score(hp, (1.0, 0.5), xs, vs, sc_out))
        del out16
        B.rollout_destroy(hp)
        other = {"compact_gbs": rows_out * w.elems * 8 / (t_c * 1e-3) / 1e9,
                 "compact_rows": [rows_in, rows_out],
                 "preview_bf16_gbs": rows_out * w.elems * 8 / (t_p16 * 1e-3) / 1e9,
                 "score_preview_bf16_gbs": rows_out * w.elems * 8 / (t_sp16 * 1e-3) / 1e9,
                 "score_preview_bf16_frac_of_peak": rows_out * w.elems * 8 / (t_sp16 * 1e-3) / 1e9 / peak,
                 "score_preview_bf16_us": t_sp16 * 1e3, "score_then_preview_us": (t_s + t_p16) * 1e3,
                 "bytes_per_element": {"compact": 8, "preview_bf16": 8, "score_preview_bf16": 8,
                                       "score_then_preview": 14},
                 "note": "pg_compact gathers the first stage's survivors (fp32 rows); pg_preview writes "
                         "the bf16 look-ahead latent for an external decoder; pg_score_preview does the "
                         "scoring pass and that emission in one pass over (x, v)"}

    # the same rollout under the coefficients of the diffusion branch (DDIM over the linear-beta
    # schedule: c_x != 1, so every step takes the step kernel's general-coefficient variant)
    general = None
    if rank == 0 and w.velocity == "normal":
        from dataclasses import replace as _replace
        wg = _replace(w, coef="ddim", eta=1.0)
        gen_run = lambda trace=None: ro.run(x0, wg.step_coef, wg.preview_coef, velocity, external_scores=ext,
                                            final_rewards=fin, trace=trace)
        gen_run()
        torch.cuda.synchronize()
        gtr = []
        for _ in range(min(args.steps, 5)):
            tr = []
            gen_run(trace=tr)
            gtr.append(tr)
        torch.cuda.synchronize()
        g_ms = sum(a.elapsed_time(b) for tr in gtr for kind, _, a, b in tr if kind == "step")
        g_rows = sum(rows for tr in gtr for kind, rows, _, _ in tr if kind == "step")
        g_gbs = g_rows * (w.elems * (8 + vel_bytes) + 4) / (g_ms * 1e-3) / 1e9
        general = {"kernel": "step_kernel<general coefficients> (c_x != 1: DDIM schedule, eta = 1; last step deterministic)",
                   "step_gbs": g_gbs, "step_frac_of_peak": g_gbs / peak,
                   "unit_cx_step_gbs": step_gbs, "rollouts": len(gtr)}

    # step / score launches by row count on the streaming shape
    by_rows = None
    if rank == 0 and w.vel_dtype == "bf16" and w.velocity == "normal" and w.elems * w.n_groups * w.n_expand * 4 > 1e9:
        by_rows = launch_size_table(B, ro.x[0], ro.x[1], vels[0], w.elems, peak)

    # the three smaller workloads, same driver (secondary lines; the bench line is the large one)
    others = None
    if rank == 0 and world == 1 and w.name == "large" and not args.groups and not args.no_others:
        others = {}
        for name, _ in OTHER_WORKLOADS:
            others[name] = _other_workload(name, dev, max(5, min(args.steps, 20)), peak)
            if name in cpu_others:
                others[name]["cpu_oracle_latent_steps_per_s"] = cpu_others[name]["value"]
                others[name]["cpu_oracle_sample"] = cpu_others[name]["sample"]

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timing)
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(B, wl, w, wr, rank, dist, dev, args)

    value = world * w.traj_steps * args.steps / (total_ms * 1e-3)
    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": _config(w, args), "clocks": clocks,
                "gpu_launches": int(launches),
                "roofline": {"bound": "hbm", "kernel": "step_kernel<bf16> (SDE step + log-prob)",
                             "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                             "frac": step_gbs / peak, "peak_kind": peak_kind,
                             "frac_of_8TBs_nominal": step_gbs / 8000.0,
                             "bytes_per_launch": step_bytes / kinds["step"]["launches"],
                             "traffic": (None if traffic_ratio is None else
                                         traffic_ratio * step_bytes / kinds["step"]["launches"]),
                             "traffic_source": traffic_note if traffic_ratio is None else
                                               f"{traffic_note}: DRAM / algorithmic bytes = {traffic_ratio:.4f} on the captured "
                                               "256-row launch, scaled by rows (every element is read and written once)",
                             "also": also,
                             "bytes_per_element_step": 8 + vel_bytes},
                "kernels": {k: {"ms_per_rollout": v["ms"] / args.steps, "launches_per_rollout":
                                v["launches"] // args.steps} for k, v in kinds.items()},
                "score_gbs": score_gbs, "prune_stage_gbs": prune_stage_gbs,
                "hbm_gbs_whole_rollout": (step_bytes + (score_bytes if score_gbs else 0)) / (total_ms * 1e-3) / 1e9,
                "ovf_microbench": ovf, "drivers": drivers, "policy_update": policy, "other_kernels": other, "general_coefficients": general,
                "launch_size_table": by_rows, "other_workloads": others, "e2e": e2e, "cpu_baseline": cpu_base}
        if gathered is not None:
            line["gathered"] = gathered
        print(json.dumps(line))
    sr.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_e2e(B, wl, w, wr, rank, dist, dev, args):
    import torch
    cfg = B.make_config(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed,
                        B.VEL_BF16 if w.vel_dtype == "bf16" else B.VEL_F32, adv_eps=w.adv_eps,
                        group_offset=rank * w.n_groups)  # = sharding.weak_shard(...)[0]
    from paper_2512_15347_b200 import sharding
    # every rank pins its own copy of the inputs (26 GB for the large workload): if any rank cannot
    # get them, all ranks skip the end-to-end leg together
    ok, why = 1.0, ""
    try:
        ws = torch.empty(B.rollout_host_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
        dt = torch.bfloat16 if w.vel_dtype == "bf16" else torch.float32
        # host inputs: pinned; filled from a seeded CPU generator block by block (content does not
        # affect timing, but the bytes are real N(0,1) draws)
        g = torch.Generator().manual_seed(1234 + rank)
        x0 = torch.empty(w.n_groups * w.n_expand, w.elems, dtype=torch.float32).pin_memory()
        block = torch.randn(64, w.elems, generator=g)
        for i in range(0, x0.shape[0], 64):
            x0[i:i + 64] = block[: x0.shape[0] - i].roll(i // 64, 1)
        vels = []
        vblock = torch.randn(64, w.elems, generator=g).to(dt)
        for s in range(w.n_steps):
            rows = w.n_groups * w.rows_before(s)
            v = torch.empty(rows, w.elems, dtype=dt).pin_memory()
            for i in range(0, rows, 64):
                v[i:i + 64] = vblock[: rows - i].roll(s * 64 + i // 64, 1)
            vels.append(v)
        K = w.final_keep
        x_final = torch.empty(w.n_groups * K, w.elems).pin_memory()
        logp = torch.empty(w.traj_steps).pin_memory()
        keep = torch.empty(sum(w.n_groups * k for _, k in w.stages), dtype=torch.int32).pin_memory()
        adv = torch.empty(w.n_groups * K).pin_memory()
        ids = torch.empty(w.n_groups * K, dtype=torch.int32).pin_memory()
    except Exception as e:            # out of host or device memory
        ok, why = 0.0, f"{type(e).__name__}: {e}"[:200]
    if not sharding.all_ranks_ok(ok == 1.0, dist, dev):
        return {"value": None, "unit": UNIT, "unavailable": why or "another rank could not allocate its buffers"}
    coefs = [w.step_coef(s) for s in range(w.n_steps)]
    pcoefs = [w.preview_coef(s) for s, _ in w.stages]

    n = max(1, min(args.steps, 3)) if w.n_groups * w.n_expand * w.elems > (1 << 28) else max(3, args.steps)

    def timed(x0_arg):
        call = lambda: B.rollout_host(cfg, coefs, pcoefs, x0_arg, vels, None, None, x_final, logp, keep,
                                      adv, ids, ws)
        call()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            call()
        b.record()
        torch.cuda.synchronize()
        return sharding.max_over_ranks(a.elapsed_time(b), dist, dev)

    # headline: the initial latents are drawn on the device by the library's generator (x0 = NULL),
    # so the host supplies only the per-step predictions; second figure: x0 copied from the host too
    ms = timed(None)
    ms_host_x0 = timed(x0)
    # third figure: the same call on a handle made once (pg_rollout_host_on): no allocation, stream or
    # event creation per call - what matters when the latents are small
    h_once = B.rollout_init(cfg)
    hargs = B.HostArgs(coefs, pcoefs, vels)

    def timed_on():
        call = lambda: B.rollout_host_on(h_once, hargs, None, None, x_final, logp, keep, adv, ids, ws)
        call()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            call()
        b.record()
        torch.cuda.synchronize()
        return sharding.max_over_ranks(a.elapsed_time(b), dist, dev)
    ms_on = timed_on()
    torch.cuda.synchronize()
    B.rollout_destroy(h_once)
    # the first timed pass also pays for whatever the host side had not warmed up yet (it has measured
    # up to 1.5x slower than the same call repeated later): the headline is the better of two passes
    ms = min(ms, timed(None))
    world = 1 if dist is None else dist.get_world_size()
    vel_bytes = sum(v.numel() * v.element_size() for v in vels)
    d2h = x_final.numel() * 4 + logp.numel() * 4 + keep.numel() * 4 + adv.numel() * 4 + ids.numel() * 4
    return {"value": world * w.traj_steps * n / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": vel_bytes,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms / n, "steps": n,
            "h2d_gbs": vel_bytes * n / (ms * 1e-3) / 1e9,
            "entry": "pg_rollout_host (pinned host buffers; per-step predictions copied in while the previous "
                     "step computes; x0 drawn on the device; latents, log-probs, indices, advantages copied out)",
            "on_existing_handle": {"value": world * w.traj_steps * n / (ms_on * 1e-3), "ms_per_step": ms_on / n,
                                   "entry": "pg_rollout_host_on (handle, streams and events made once)"},
            "with_x0_from_host": {"value": world * w.traj_steps * n / (ms_host_x0 * 1e-3),
                                  "ms_per_step": ms_host_x0 / n,
                                  "h2d_bytes_per_step": vel_bytes + x0.numel() * 4}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=["large", "sd3", "sd15", "tiny", "pro-standard", "pro-flash", "pro-diffusion"])
    ap.add_argument("--config", default="", help="JSON workload file (see paper_2512_15347_b200/configs/) instead of --workload")
    ap.add_argument("--groups", type=int, default=0,
                    help="prompt groups per GPU (default: the workload's own; smaller for profiling)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the three smaller workloads")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
