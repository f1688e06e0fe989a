"""CUDA path vs the fp64 oracle, element by element, through the C ABI (needs a GPU)."""
import numpy as np
import pytest
import torch

from oracle import run as orun
from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}   # max over l of ||g_l - oracle|| / ||oracle||


def rel_l2(a, b):
    b = np.asarray(b, dtype=np.float64)
    a = np.asarray(a, dtype=np.float64).reshape(b.shape)
    nb = np.linalg.norm(b)
    if nb == 0.0:  # an all-zero reference (the RNN's initial state) must be matched exactly
        return float(np.linalg.norm(a))
    return float(np.linalg.norm(a - b) / nb)


def to_np(t):
    return t.detach().float().cpu().double().numpy()


def run_gpu(w, inp, ks, want_grads=True):
    from paper_2501_17086_b200 import harness
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    xin = harness.rnn_inputs(w, inp)
    x_all = ctx.forward(params, inp["x0"], xin)
    delta = harness.loss_delta(w, x_all, inp)
    out = {"x": x_all, "hbp": {}, "grads": {}, "ctx": ctx}
    for k in ks:
        grads = ctx.new_grads(with_gate=True) if want_grads else None
        out["hbp"][k] = ctx.backward(params, k, delta, x_all, xin, grads=grads).clone()
        out["grads"][k] = grads
    grads = ctx.new_grads(with_gate=True) if want_grads else None
    out["exact"] = ctx.exact(params, delta, x_all, xin, grads=grads)
    out["grads"]["exact"] = grads
    ctx.sync_status()
    return out


def compare(w, gpu, ref, ks, grads_for):
    tol = TOL[w.dtype]
    steps = w.steps
    shape = ref["xs"][0].shape
    for l in range(steps + 1):
        assert rel_l2(to_np(gpu["x"][l]), ref["xs"][l]) < tol, f"state {l}"
    def worst_over_states(got, want):
        """Max per-state rel-L2.  A state whose exact value lies below the normal range of float (products of many
        gates below one, with a loss on the last state only) cannot be held to a relative bound: it only has to be
        as small on the GPU."""
        floor = 1e-30 * max(np.linalg.norm(r) for r in want)
        worst = 0.0
        for l in range(steps + 1):
            if np.linalg.norm(want[l]) < floor:
                assert np.linalg.norm(to_np(got[l])) <= floor, f"state {l} should have vanished"
            else:
                worst = max(worst, rel_l2(to_np(got[l]), want[l]))
        return worst

    for k in ks:
        worst = worst_over_states(gpu["hbp"][k], ref["hbp"][k])
        assert worst < tol, f"k={k}: max rel-L2 {worst:.3e}"
    worst = worst_over_states(gpu["exact"], ref["exact"])
    assert worst < tol, f"exact: max rel-L2 {worst:.3e}"
    for key in grads_for:
        for name, val in ref["grads"][key].items():
            got = gpu["grads"][key]["d" + name]
            e = rel_l2(to_np(got), val)
            assert e < tol, f"grad {name} ({key}): rel-L2 {e:.3e}"


@pytest.mark.parametrize("name,ks", [
    ("c1", tuple(range(0, 10))),
    ("c2_twin_f32", (0, 1, 2, 5, 7)),
    ("c2_twin", (0, 1, 2, 4, 5)),
    ("c5_twin", (1, 3, 9)),
    ("c3_twin", (0, 1, 2, 4, 8)),
    ("c4_twin_f32", (0, 1, 2, 4)),
    ("c4_twin", (1, 2, 4)),
    ("gru_twin", (0, 1, 2, 4, 8, 40)),
    ("gru_twin_long", (0, 1, 3)),
    ("gru_twin_bf16", (1, 2, 4)),
    ("lstm_twin", (0, 1, 2, 4, 8, 40)),
    ("lstm_twin_long", (0, 1, 3)),
    ("lstm_twin_bf16", (1, 2, 4)),
    ("relu_twin", (0, 1, 2, 5)),
    ("postln_twin", (0, 1, 2, 5)),
    ("postln_twin_bf16", (1, 2, 5)),
    ("postln_twin_shift", (0, 1, 2, 5)),
    ("postln_twin_shift_bf16", (1, 2, 6)),
])
def test_twin_matches_oracle_in_full(name, ks):
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    gpu = run_gpu(w, inp, ks)
    kmax = max(ks)
    ref = orun.run(w, inp, ks=ks, grads_for=("exact", kmax))
    compare(w, gpu, ref, ks, ("exact", kmax))
    # k >= steps is the exact gradient (Theorem 2), also on the GPU
    if kmax >= w.steps:
        for l in range(w.steps + 1):
            assert rel_l2(to_np(gpu["hbp"][kmax][l]), to_np(gpu["exact"][l])) < TOL[w.dtype]


def test_runs_are_bitwise_reproducible():
    w = WORKLOADS["c2_twin"]
    inp = make_inputs(w, "cuda")
    a = run_gpu(w, inp, (2,))
    b = run_gpu(w, inp, (2,))
    assert torch.equal(a["hbp"][2], b["hbp"][2])
    for n in a["grads"][2]:
        assert torch.equal(a["grads"][2][n], b["grads"][2][n])
