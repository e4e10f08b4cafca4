"""The C-ABI library loads on a machine without a GPU and exports every declared entry point;
argument validation that precedes any CUDA call works there too."""
import ctypes
import os
import re

import pytest

from paper_2512_15347_b200 import binding as B
from paper_2512_15347_b200 import build as pg_build
from paper_2512_15347_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pg_build.build()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "progrpo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pg_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"pg_rollout_init", "pg_step", "pg_score", "pg_prune_ovf", "pg_compact", "pg_advantages",
            "pg_ovf_select_batched", "pg_rollout_host"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_error_strings(lib):
    for code in (0, -1, -2, -3, -4, -5, -6, -7, -8, -9):
        assert B.strerror(code) and "unknown" not in B.strerror(code)
    assert "unknown" in B.strerror(-99)


@pytest.mark.parametrize("kw", [
    dict(n_groups=0), dict(n_expand=0), dict(n_expand=B.MAX_GROUP + 1), dict(elems=6), dict(elems=0),
    dict(n_steps=0), dict(stages=[(3, 8), (3, 4)]), dict(stages=[(3, 8), (2, 4)]),
    dict(stages=[(3, 17)]), dict(stages=[(3, 8), (5, 9)]), dict(stages=[(10, 8)]),
    dict(stages=[(3, 0)]), dict(vel_dtype=7), dict(adv_eps=-1.0), dict(group_offset=-1),
    dict(group_offset=2**31 - 2),
])
def test_bad_schedules_are_rejected_before_any_cuda_call(lib, kw):
    base = dict(n_groups=1, n_expand=16, elems=4096, n_steps=10, stages=[(3, 8)], seed=0,
                vel_dtype=B.VEL_F32, group_offset=0, adv_eps=1e-6)
    base.update(kw)
    cfg = B.make_config(base["n_groups"], base["n_expand"], base["elems"], base["n_steps"],
                        base["stages"], base["seed"], base["vel_dtype"],
                        group_offset=base["group_offset"], adv_eps=base["adv_eps"])
    with pytest.raises(B.PgError) as e:
        B.rollout_init(cfg)
    assert e.value.code == B.EINVAL
    assert B.rollout_host_workspace_bytes(cfg) == 0


def test_null_arguments(lib):
    assert lib.pg_rollout_init(None, None) == B.EINVAL
    assert lib.pg_rollout_destroy(None) == B.OK
    assert lib.pg_ovf_select_batched(1, 8, 9, None, None, None, None, 1e-6, None, None) == B.EINVAL
    assert lib.pg_ovf_select_batched(1, 2048, 9, None, None, None, None, 1e-6, None, None) == B.EINVAL


def test_workspace_size_covers_the_large_workload(lib):
    w = wl.WORKLOADS["large"]
    cfg = B.make_config(w.n_groups, w.n_expand, w.elems, w.n_steps, w.stages, w.seed, B.VEL_BF16)
    need = B.rollout_host_workspace_bytes(cfg)
    rows = w.n_groups * w.n_expand
    assert need >= 2 * rows * w.elems * 4 + 2 * rows * w.elems * 2
    assert need < 2 * rows * w.elems * 4 + 2 * rows * w.elems * 2 + (1 << 22)


def test_workload_shapes_match_the_stated_totals():
    assert wl.WORKLOADS["tiny"].traj_steps == 104
    assert wl.WORKLOADS["sd15"].traj_steps == 2304
    assert wl.WORKLOADS["sd3"].traj_steps == 7680
    assert wl.WORKLOADS["large"].traj_steps == 37888
    assert wl.WORKLOADS["large"].score_rows == 4096 + 2048 + 1024
    assert wl.WORKLOADS["large"].element_steps == 37888 * 262144
