"""hbp_cumsumprod_static: the scan entry point for hosts that may not allocate device memory (their pool was
handed out at start-up, or allocation calls are forbidden while they run).  Its scratch is a fixed array in
the library.  The scratch is only used by the time-chunked form of the scan, which runs when the gate is a
table with one vector per step, so those are the cases here.  Each is checked against the oracle's sequential
recurrence (and against hbp_cumsumprod with caller-provided scratch), twice in a row with different data and
once after a larger problem, so the second and third calls find leftovers in the shared array.  A problem
beyond the fixed size must be refused.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import hbp_oracle as O

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2}


def _case(seed, L, rows, d, dtype):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    u = torch.randn((L, rows, d), generator=gen, device="cuda").to(dtype)
    delta = torch.randn((L + 1, rows, d), generator=gen, device="cuda").to(dtype)
    a = (0.9 + 0.099 * torch.rand((L, d), generator=gen, device="cuda")).to(dtype)   # one gate vector per step
    return u, delta, a


def _np64(t):
    return t.detach().float().cpu().double().numpy()


def _oracle(u, delta, a):
    """Eq. 9 solved in order on v_l = u_l + delta_l with the carry delta_L beyond the last step."""
    L = u.shape[0]
    dl = _np64(delta)
    v = [_np64(u[l]) + dl[l] for l in range(L)] + [dl[L]]
    gates = [_np64(a[l]) for l in range(L)] + [1.0]
    return np.stack(O.cumsumprod_sequential(v, gates))


def _worst(got, ref):
    g = _np64(got)
    return max(float(np.linalg.norm(g[l] - ref[l]) / np.linalg.norm(ref[l])) for l in range(ref.shape[0]))


def _check(seed, L, rows, d, dtype, g_out=None):
    from paper_2501_17086_b200 import binding as B
    need = B.cumsumprod_scratch_bytes(dtype, L, rows, d)
    assert 0 < need <= B.cumsumprod_static_max_bytes()       # the chunked form, within the fixed array
    u, delta, a = _case(seed, L, rows, d, dtype)
    ref = _oracle(u, delta, a)
    got = B.cumsumprod_static(u, delta, a, gate=B.GATE_CHANNEL_PER_STEP, loss=B.LOSS_EVERY_STEP, g=g_out)
    torch.cuda.synchronize()
    assert torch.isfinite(got).all()
    assert _worst(got, ref) <= TOL[dtype]
    want = B.cumsumprod(u, delta, a, gate=B.GATE_CHANNEL_PER_STEP, loss=B.LOSS_EVERY_STEP)
    torch.cuda.synchronize()
    assert _worst(got, _np64(want)) <= TOL[dtype]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_scratch_scan_matches_the_recurrence_on_repeated_calls(dtype):
    L, rows, d = 600, 8, 256
    g_out = torch.empty((L + 1, rows, d), dtype=dtype, device="cuda")    # outputs come from the caller
    for seed in (11, 12):              # second call: different data, same shared scratch
        _check(seed, L, rows, d, dtype, g_out)
    _check(13, 1500, 16, 512, dtype)   # a larger problem fills more of the array ...
    _check(14, L, rows, d, dtype, g_out)   # ... and the small one afterwards finds its leftovers
    _check(15, 257, 2, 32, dtype)      # ragged last chunk


def test_static_scratch_scan_with_a_shared_gate():
    """One gate vector for all steps: served without touching the scratch, same entry point."""
    from paper_2501_17086_b200 import binding as B
    L, rows, d = 512, 4, 128
    u, delta, a = _case(16, L, rows, d, torch.float32)
    a = a[0].contiguous()
    dl = _np64(delta)
    v = [_np64(u[l]) + dl[l] for l in range(L)] + [dl[L]]
    ref = np.stack(O.cumsumprod_sequential(v, [_np64(a)] * L + [1.0]))
    got = B.cumsumprod_static(u, delta, a, loss=B.LOSS_EVERY_STEP)
    torch.cuda.synchronize()
    assert _worst(got, ref) <= 1e-5


def test_static_scratch_scan_refuses_oversized_problem():
    from paper_2501_17086_b200 import binding as B
    L, rows, d = 8192, 32, 512          # needs 64 MiB of scratch in double
    assert B.cumsumprod_scratch_bytes(torch.float32, L, rows, d) > B.cumsumprod_static_max_bytes()
    u = torch.zeros((L, rows, d), device="cuda")
    delta = torch.zeros((rows, d), device="cuda")
    with pytest.raises(B.HbpError) as info:
        B.cumsumprod_static(u, delta)
    assert info.value.code == 5
