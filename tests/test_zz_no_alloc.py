"""pg_score_static, the scoring call for callers that may not allocate device memory (code
hosted inside another framework's memory pool, services with a fixed device footprint,
latency-critical sections): it must give what pg_score gives, call after call, although all
of its calls share one built-in scratch array that is never cleared between processes' calls
except by the entry point itself.  Collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bf16", [True, False])
def test_static_score_equals_handle_score_twice_in_a_row(bf16):
    from paper_2512_15347_b200 import binding as B
    B.lib()
    G, N0, d = 4, 24, 3 * 8192 + 20          # several chunks per row and a ragged tail
    n = G * N0
    vd = B.VEL_BF16 if bf16 else B.VEL_F32
    h = B.rollout_init(B.make_config(G, N0, d, 4, [], 5, vd))
    try:
        for call in range(2):                  # the second call meets the first one's leftovers
            g = torch.Generator(device="cuda").manual_seed(100 + call)
            x = torch.randn(n, d, device="cuda", generator=g) + 0.25 * call
            v = torch.randn(n, d, device="cuda", generator=g)
            v = v.to(torch.bfloat16) if bf16 else v
            rows = n if call == 0 else n - 7   # fewer rows the second time
            want = torch.empty(n, device="cuda")
            got = torch.full((n,), float("nan"), device="cuda")
            B.score(h, (1.0, 0.6), x, v, want)
            B.score_static(rows, d, vd, (1.0, 0.6), x, v, got)
            torch.cuda.synchronize()
            # same kernel, same reduction order: the tests' score tolerance is 1e-6 absolute
            assert np.abs(got[:rows].cpu().numpy() - want[:rows].cpu().numpy()).max() <= 1e-6
            assert torch.isnan(got[rows:]).all()
            B.score_static(rows, d, vd, (1.0, 0.0), x, None, got)
            B.score(h, (1.0, 0.0), x, None, want)
            torch.cuda.synchronize()
            assert np.abs(got[:rows].cpu().numpy() - want[:rows].cpu().numpy()).max() <= 1e-6
    finally:
        torch.cuda.synchronize()
        B.rollout_destroy(h)


def test_static_score_refuses_what_does_not_fit():
    from paper_2512_15347_b200 import binding as B
    x = torch.zeros(8, 64, device="cuda")
    out = torch.empty(8, device="cuda")
    with pytest.raises(B.PgError) as e:
        B.score_static(B.STATIC_MAX_ROWS + 1, 64, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.ECAPACITY
    with pytest.raises(B.PgError) as e:       # rows fit, rows x chunks does not
        B.score_static(B.STATIC_MAX_ROWS, 32768 * 8 + 4, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.ECAPACITY
    with pytest.raises(B.PgError) as e:
        B.score_static(8, 66, B.VEL_F32, (1.0, 0.0), x, None, out)
    assert e.value.code == B.EINVAL
    B.score_static(8, 64, B.VEL_F32, (1.0, 0.0), x, None, out)   # still usable afterwards
    torch.cuda.synchronize()
    assert torch.equal(out, torch.zeros(8, device="cuda"))
