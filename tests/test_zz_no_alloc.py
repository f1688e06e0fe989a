"""hbp_cumsumprod_static: the scan entry point for hosts that may not allocate device memory (their pool was
handed out at start-up, or allocation calls are forbidden while they run).  Its scratch is a fixed array in
the library, so this test only checks that it computes what hbp_cumsumprod computes with caller-provided
scratch, twice in a row (the second call finds the first call's leftovers in the shared array), and that a
problem beyond the fixed size is refused.  Collected last on purpose."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(seed, L, rows, d, dtype):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    u = torch.randn((L, rows, d), generator=gen, device="cuda").to(dtype)
    delta = torch.randn((L + 1, rows, d), generator=gen, device="cuda").to(dtype)
    a = (0.9 + 0.099 * torch.rand((d,), generator=gen, device="cuda")).to(dtype)
    return u, delta, a


def test_static_scratch_scan_matches_caller_scratch_scan_twice():
    from paper_2501_17086_b200 import binding as B
    L, rows, d = 600, 8, 256
    assert 0 < B.cumsumprod_scratch_bytes(torch.float32, L, rows, d) <= B.cumsumprod_static_max_bytes()
    g_out = torch.empty((L + 1, rows, d), dtype=torch.float32, device="cuda")   # outputs come from the caller
    for seed in (11, 12):   # second call: different data, same shared scratch
        u, delta, a = _case(seed, L, rows, d, torch.float32)
        want = B.cumsumprod(u, delta, a, loss=B.LOSS_EVERY_STEP)
        got = B.cumsumprod_static(u, delta, a, loss=B.LOSS_EVERY_STEP, g=g_out)
        torch.cuda.synchronize()
        err = (got.double() - want.double()).norm() / want.double().norm()
        assert float(err) <= 1e-5, float(err)
        assert torch.isfinite(got).all()
    # bf16 data, float scratch
    u, delta, a = _case(13, 512, 4, 128, torch.bfloat16)
    want = B.cumsumprod(u, delta, a, loss=B.LOSS_EVERY_STEP)
    got = B.cumsumprod_static(u, delta, a, loss=B.LOSS_EVERY_STEP)
    torch.cuda.synchronize()
    assert float((got.double() - want.double()).norm() / want.double().norm()) <= 2e-2


def test_static_scratch_scan_refuses_oversized_problem():
    from paper_2501_17086_b200 import binding as B
    L, rows, d = 8192, 32, 512          # needs 64 MiB of scratch in double
    assert B.cumsumprod_scratch_bytes(torch.float32, L, rows, d) > B.cumsumprod_static_max_bytes()
    u = torch.zeros((L, rows, d), device="cuda")
    delta = torch.zeros((rows, d), device="cuda")
    with pytest.raises(B.HbpError) as info:
        B.cumsumprod_static(u, delta)
    assert info.value.code == 5
