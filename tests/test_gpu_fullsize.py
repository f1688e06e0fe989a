"""Full-size workloads on the GPU, in the launch configuration the benchmark times, checked against the
fp64 oracle on sampled independent units (tokens / sequences / batch rows): the blocks act on each unit
independently, so the oracle run on a subset with the full weights gives exactly those rows of every g_l."""
import numpy as np
import pytest
import torch

from oracle import run as orun
from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}
# Exact BPTT on c3 is ill-conditioned: with a in U(0.9, 0.999) plus 0.5 x orthogonal recurrent weights the step
# Jacobian a + tanh'(z) W has growth ~1.007 per step, so ||g_0|| / ||g_T|| ~ 1e13 over 4096 steps and the float
# rounding of the stored states (2.6e-7 between the two forward passes) is amplified through hundreds of
# factors.  Highway-BP with k <= 8 applies at most 8 block Jacobians and keeps the 1e-5 bar; exact BPTT at the
# full length is held to this looser bound (it meets 1e-5 on the T = 200 twin).
TOL_EXACT_LONG_RNN = 5e-4


def _rows_of(w, t, rows):
    """[steps+1, N, d] -> the sampled units, shaped like the oracle's states."""
    if w.block == "preln_transformer":
        return t.reshape(t.shape[0], w.batch, w.seq, w.d)[:, rows]
    return t[:, rows]


@pytest.mark.parametrize("name,ks,rows", [
    ("c2", (1, 2, 4, 8), [0, 1, 127, 128, 4097, 8191]),
    ("c3", (1, 2, 4, 8), [0, 31]),
    ("c4", (1, 2, 4), [5]),
    ("c5", (1, 2), [0, 129, 8200, 16383]),
    ("g1", (1, 2, 4), [0, 77, 127]),
    ("g2", (1, 3, 8), [0, 1, 64, 127]),
    ("l1", (1, 2, 4), [0, 77, 127]),
    ("p2", (1, 2, 4), [0, 1, 127, 128, 4097, 8191]),
])
def test_full_size_sampled_units(name, ks, rows):
    from paper_2501_17086_b200 import harness
    w = WORKLOADS[name]
    need_gb = {"c2": 30, "c3": 4, "c4": 40, "c5": 150, "g1": 4, "g2": 1, "l1": 6, "p2": 34}[name]
    free, _ = torch.cuda.mem_get_info()
    if free < need_gb * 2**30:
        pytest.skip(f"needs about {need_gb} GB of free device memory")
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    xin = harness.rnn_inputs(w, inp)
    x_all = ctx.forward(params, inp["x0"], xin)
    delta = harness.loss_delta(w, x_all, inp)
    rows_t = torch.tensor(rows, device="cuda")
    got = {}
    g_all = ctx.new_states()
    for k in ks:
        ctx.backward(params, k, delta, x_all, xin, g_all=g_all)
        got[k] = _rows_of(w, g_all, rows_t).float().cpu().double().numpy()
    grads = ctx.new_grads(with_gate=True)
    ctx.exact(params, delta, x_all, xin, g_all=g_all, grads=grads)
    got["exact"] = _rows_of(w, g_all, rows_t).float().cpu().double().numpy()
    ctx.sync_status()
    xs_gpu = _rows_of(w, x_all, rows_t).float().cpu().double().numpy()
    for t in grads.values():
        assert torch.isfinite(t).all()
    del ctx, g_all, x_all, grads
    torch.cuda.empty_cache()

    ref = orun.run(w, inp, ks=ks, rows=rows_t.cpu())
    tol = TOL[w.dtype]

    def rel(a, b):
        nb = np.linalg.norm(b)
        return float(np.linalg.norm(a.reshape(b.shape) - b) / nb) if nb else float(np.linalg.norm(a))

    worst_x = max(rel(xs_gpu[l], ref["xs"][l]) for l in range(w.steps + 1))
    assert worst_x < tol, f"states: {worst_x:.3e}"

    def worst_over_states(got_k, ref_k):
        """Max per-state rel-L2; a state whose exact value lies below the range of float (a shifted split scales
        each state by (1 - gamma) per step: 0.2^64 on p2) only has to be as small on the GPU."""
        floor = 1e-30 * max(np.linalg.norm(r) for r in ref_k)
        worst = 0.0
        for l in range(w.steps + 1):
            if np.linalg.norm(ref_k[l]) < floor:
                assert np.linalg.norm(got_k[l]) <= floor, f"state {l} should have vanished"
            else:
                worst = max(worst, rel(got_k[l], ref_k[l]))
        return worst

    for k in ks:
        worst = worst_over_states(got[k], ref["hbp"][k])
        assert worst < tol, f"k={k}: max rel-L2 {worst:.3e}"
    worst = max(rel(got["exact"][l], ref["exact"][l]) for l in range(w.steps + 1))
    tol_exact = TOL_EXACT_LONG_RNN if name == "c3" else tol
    assert worst < tol_exact, f"exact: max rel-L2 {worst:.3e}"
    # tail exactness on the GPU itself (Theorem 2): g^k_l is already exact for l >= steps - k
    kmax = max(ks)
    for l in range(w.steps - kmax, w.steps + 1):
        assert rel(got[kmax][l], got["exact"][l]) < tol_exact


def _run_shard(w_shard, inp, rows, delta_rows):
    """hbp_backward(k=2) with parameter gradients on the token shard `rows` of a workload (full weights)."""
    from paper_2501_17086_b200 import harness
    ctx = harness.make_context(w_shard)
    params = harness.params_for(w_shard, inp)
    x_all = ctx.forward(params, inp["x0"][rows].contiguous(), None)
    grads = ctx.new_grads()
    ctx.backward(params, 2, delta_rows, x_all, None, grads=grads)
    ctx.sync_status()
    return x_all, grads


def test_full_size_parameter_gradients_by_shard_additivity():
    """Parameter gradients are sums over tokens: on c2 the gradients of the whole batch must equal the sum of the
    gradients of its two halves (each run as its own problem with the same delta rows), and a small shard must
    match the oracle run on those tokens with the full weights."""
    import dataclasses
    from paper_2501_17086_b200 import harness
    w = WORKLOADS["c2"]
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2**30:
        pytest.skip("needs about 40 GB of free device memory")
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    x_all = ctx.forward(params, inp["x0"], None)
    delta = harness.loss_delta(w, x_all, inp)          # [N, d], normalised by the full problem size
    whole = ctx.new_grads()
    ctx.backward(params, 2, delta, x_all, None, grads=whole)
    ctx.sync_status()
    del ctx, x_all
    torch.cuda.empty_cache()

    half = w.tokens // 2
    w_half = dataclasses.replace(w, tokens=half, batch=w.batch // 2)
    total = None
    for lo in (0, half):
        rows = torch.arange(lo, lo + half, device="cuda")
        _, g = _run_shard(w_half, inp, rows, delta[rows].contiguous())
        total = g if total is None else {n: total[n] + g[n] for n in g}
        torch.cuda.empty_cache()
    for n in whole:
        err = float((whole[n].double() - total[n].double()).norm() / total[n].double().norm())
        assert err < 2e-3, f"{n}: whole vs sum of halves {err:.3e}"   # same bf16 products, other summation order

    # a 48-token shard against the oracle (tokens are independent, so its delta rows are the whole problem's)
    rows = torch.tensor([0, 1, 2, 3, 130, 131, 4099, 8191] + list(range(1000, 1040)), device="cuda")
    w_small = dataclasses.replace(w, tokens=int(rows.numel()), batch=1, seq=int(rows.numel()))
    x_small, g_small = _run_shard(w_small, inp, rows, delta[rows].contiguous())
    stack, x0, groups = orun.build_stack(w, inp, rows.cpu())
    from oracle import hbp_oracle as O
    xs, caches = O.forward(stack, x0)
    deltas = orun.loss_deltas(w, xs, inp, rows.cpu())
    gk = O.highway_bp(stack, caches, deltas, 2)
    ref = O.param_grads(stack, caches, xs, gk, groups)
    for n, v in ref.items():
        got = g_small["d" + n].double().cpu().numpy()
        err = float(np.linalg.norm(got - v) / np.linalg.norm(v))
        assert err < TOL[w.dtype], f"{n}: shard vs oracle {err:.3e}"
