"""The plain C example builds against include/progrpo.h and the shared library; on a GPU it runs
a small rollout without Python in the loop."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PKG = os.path.join(ROOT, "paper_2512_15347_b200")
SRC = os.path.join(PKG, "examples", "abi_example.c")


def _build(tmp_path):
    exe = str(tmp_path / "abi_example")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    cmd = ["gcc", "-std=c11", "-Wall", "-Werror", SRC, "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(cuda, "include"), "-L", PKG, "-lprogrpo", "-L", os.path.join(cuda, "lib64"),
           "-lcudart", "-lm", "-o", exe]
    subprocess.run(cmd, check=True)
    return exe


def test_c_example_compiles_and_links(tmp_path):
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
def test_c_example_runs(tmp_path):
    exe = _build(tmp_path)
    env = dict(os.environ, LD_LIBRARY_PATH=PKG + ":" + os.environ.get("LD_LIBRARY_PATH", ""))
    res = subprocess.run([exe], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "group 1 advantages" in res.stdout and "kernel launches" in res.stdout
