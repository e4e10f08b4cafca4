"""pg_score_static, the scoring call for callers that may not allocate device memory (code
hosted inside another framework's memory pool, services with a fixed device footprint,
latency-critical sections).  Its reduction scratch is one array built into the library, shared
by all calls on a device and never cleared except by the entry point itself, so the checks here
are made on several calls in a row: each call meets what the previous one left in the array
(partial sums of other rows, counters of a different row count or a different number of
partial sums per row).  Every call is compared with the CPU oracle and with pg_score.
Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_15347_b200 import workloads as wl
from tests import util as U

pytestmark = pytest.mark.gpu

STATIC_CHUNK = 32768          # elements per partial sum of pg_score_static (documented in progrpo.h)


def _check_call(B, h_by_d, rows, d, bf16, seed, coef):
    """One pg_score_static call on fresh data against the oracle and against pg_score."""
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((rows, d)) + 0.25 * (seed % 3)).astype(np.float32)
    vt = torch.from_numpy(rng.standard_normal((rows, d)).astype(np.float32))
    vt = vt.to(torch.bfloat16) if bf16 else vt
    v = wl.as_numpy_velocity(vt)
    vd = B.VEL_BF16 if bf16 else B.VEL_F32
    x_dev, v_dev = U.to_dev(x), U.vel_to_dev(v)
    got = torch.full((rows + 5,), float("nan"), device="cuda")
    use_vel = coef[1] != 0.0
    B.score_static(rows, d, vd, coef, x_dev, v_dev if use_vel else None, got)
    torch.cuda.synchronize()
    got_np = got.cpu().numpy()
    ref = oracle.score(x, v, coef[0], coef[1])[0]
    assert np.abs(got_np[:rows] - ref).max() <= U.SCORE_GAP
    assert np.isnan(got_np[rows:]).all()                      # nothing written past the rows asked for
    # the handle-based call on the same rows (its own scratch, shorter chunks): same tolerance
    G, N0, h = h_by_d[d]
    if rows == G * N0:
        want = torch.empty(rows, device="cuda")
        B.score(h, coef, x_dev, v_dev if use_vel else None, want)
        torch.cuda.synchronize()
        assert np.abs(got_np[:rows] - want.cpu().numpy()).max() <= U.SCORE_GAP


@pytest.mark.parametrize("bf16", [True, False])
def test_static_score_matches_oracle_call_after_call(bf16):
    from paper_2512_15347_b200 import binding as B
    B.lib()
    d_ragged = 3 * STATIC_CHUNK + 20         # 4 partial sums per row, the last one over 20 elements
    d_even = 8 * STATIC_CHUNK                # 8 partial sums per row (the 16x128x128 latent)
    assert -(-d_ragged // STATIC_CHUNK) == 4 and d_even // STATIC_CHUNK == 8
    vd = B.VEL_BF16 if bf16 else B.VEL_F32
    handles = {d_ragged: (4, 24, B.rollout_init(B.make_config(4, 24, d_ragged, 4, [], 5, vd))),
               d_even: (2, 6, B.rollout_init(B.make_config(2, 6, d_even, 4, [], 5, vd)))}
    try:
        # two calls in a row on the same shape, then fewer rows (the first call's partial sums of
        # the rows beyond stay in the array), then another number of partial sums per row (the
        # slots are laid out differently), then the first shape again, then the mean of x alone
        _check_call(B, handles, 96, d_ragged, bf16, 1, (1.0, 0.6))
        _check_call(B, handles, 96, d_ragged, bf16, 2, (1.0, 0.6))
        _check_call(B, handles, 89, d_ragged, bf16, 3, (0.7, -0.4))
        _check_call(B, handles, 12, d_even, bf16, 4, (1.0, 0.25))
        _check_call(B, handles, 96, d_ragged, bf16, 5, (1.0, 0.6))
        _check_call(B, handles, 96, d_ragged, bf16, 6, (1.0, 0.0))
    finally:
        torch.cuda.synchronize()
        for _, _, h in handles.values():
            B.rollout_destroy(h)


def test_static_score_refuses_what_does_not_fit():
    from paper_2512_15347_b200 import binding as B
    x = torch.zeros(8, 64, device="cuda")
    out = torch.empty(8, device="cuda")
    with pytest.raises(B.PgError) as e:
        B.score_static(B.STATIC_MAX_ROWS + 1, 64, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.ECAPACITY
    with pytest.raises(B.PgError) as e:       # rows fit, rows x partial sums per row does not
        B.score_static(B.STATIC_MAX_ROWS, STATIC_CHUNK * 8 + 4, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.ECAPACITY
    with pytest.raises(B.PgError) as e:
        B.score_static(8, 66, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.EINVAL
    B.score_static(8, 64, B.VEL_F32, (1.0, 0.0), x, None, out)   # still usable afterwards
    torch.cuda.synchronize()
    assert torch.equal(out, torch.zeros(8, device="cuda"))
