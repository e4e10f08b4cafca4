"""bench.py prints one JSON line with the agreed keys: the CPU arm (the oracle, timed) is checked
here without a GPU, the GPU arm on a small workload."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
             "scaling", "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline", "gpu_launches")


def _run(args, env_extra=None, timeout=600):
    env = dict(os.environ)
    env.update(env_extra or {})
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=timeout)
    assert p.returncode == 0, p.stderr[-2000:]
    return [ln for ln in p.stdout.splitlines() if ln.strip()]


def test_reference_arm_prints_one_line_with_the_contract_keys():
    lines = _run(["--impl", "reference", "--workload", "sd15", "--steps", "1", "--warmup", "1"])
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in BASE_KEYS:
        assert k in d, k
    assert d["impl"] == "reference" and d["unit"] == "latent-steps/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 1 and d["vs_baseline"] is None and d["dtype"] == "f64"
    assert "workload" in d["config"] and d["config"]["workload"].startswith("sd15")
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == d["value"]
    assert isinstance(cb["cpu_model"], str) and cb["cpu_model"]
    e = d["e2e"]
    assert e["value"] == d["value"] and e["unit"] == d["unit"]
    assert e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0
    assert d["gpu_launches"] == 0


def test_reference_arm_is_silent_on_other_ranks():
    assert _run(["--impl", "reference", "--workload", "sd15", "--steps", "1", "--warmup", "1"],
                {"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"}) == []


@pytest.mark.gpu
def test_gpu_arm_prints_roofline_baseline_and_end_to_end():
    lines = _run(["--workload", "sd15", "--steps", "3", "--warmup", "3"])
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in BASE_KEYS + ("roofline", "clocks"):
        assert k in d, k
    assert "impl" not in d and d["n_gpus"] == 1 and d["warmup"] >= 3 and d["dtype"] == "f32"
    assert d["value"] > 0 and d["gpu_launches"] > 0 and d["scaling"] == "weak"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["achieved"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    # the prune stage (scoring pass + selection) is in the record next to the step kernel
    stage = [a for a in r["also"] if a["kernel"].startswith("score + ovf")]
    assert len(stage) == 1 and stage[0]["achieved"] > 0 and abs(stage[0]["frac"] - stage[0]["achieved"] / r["peak"]) < 1e-9
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1 and cb["sample"] and cb["cpu_model"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] != d["value"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def _torchrun(args, timeout=600, port_offset=0):
    """One rank under the distributed launcher (rendezvous on 127.0.0.1): the process-group set-up,
    the build barrier, the max-over-ranks reduction and the gather all execute, on one GPU."""
    port = 23000 + (os.getpid() % 4000) * 2 + port_offset      # a port of its own for every launch
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "1",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    env = dict(os.environ, NCCL_NVLS_ENABLE="0")
    p = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)
    assert p.returncode == 0, (p.stdout[-1500:], p.stderr[-2500:])
    return [ln for ln in p.stdout.splitlines() if ln.strip().startswith("{")]


@pytest.mark.gpu
def test_gpu_arm_under_the_distributed_launcher():
    lines = _torchrun(["bench.py", "--gpus", "1", "--workload", "sd15", "--steps", "2", "--warmup", "3",
                       "--no-e2e", "--no-cpu-baseline"])
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 1 and d["value"] > 0 and d["gpu_launches"] > 0
    g = d["gathered"]                     # only present when a process group exists
    assert g["groups"] == 8 and g["survivors"] == 8 * 12 and g["shards"] == [[0, 8]]
    assert g["adv_abs_group_mean_max"] < 1e-5


@pytest.mark.gpu
def test_sharded_launcher_runs_and_gathers():
    lines = _torchrun(["-m", "paper_2512_15347_b200.sharded", "--workload", "sd15", "--groups", "5",
                       "--reps", "2"], port_offset=1)
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["ranks"] == 1 and d["groups"] == 5 and d["shards"] == [[0, 5]] and d["survivors"] == 5 * 12
    assert d["latent_steps_per_s"] > 0 and d["adv_abs_mean_per_group_max"] < 1e-5
    # trajectory ids are global ids of 5 groups x 24 trajectories
    assert 0 < d["traj_id_checksum"] < 5 * 12 * 5 * 24
