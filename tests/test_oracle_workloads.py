"""The oracle driven on the synthetic workloads: structure-level checks on CPU."""
import numpy as np
import pytest
import torch

from oracle import run as orun
from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs


def rel_l2(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def test_c1_full_sweep_and_empirical_error_decay():
    cfg = WORKLOADS["c1"]
    inp = make_inputs(cfg, "cpu")
    res = orun.run(cfg, inp, ks=range(0, 9), grads_for=("exact", 8))
    g = res["exact"]
    errs = [max(rel_l2(res["hbp"][k][l], g[l]) for l in range(cfg.L + 1)) for k in range(9)]
    assert errs[8] < 1e-12                      # exact once k reaches L (Theorem 2)
    for k in range(9):                          # tail exactness for l >= L-k
        for l in range(cfg.L - k, cfg.L + 1):
            assert rel_l2(res["hbp"][k][l], g[l]) < 1e-12
    for name in ("W1", "W2"):
        assert rel_l2(res["grads"][8][name], res["grads"]["exact"][name]) < 1e-12
        assert res["grads"]["exact"][name].shape == tuple(inp[name].shape)


@pytest.mark.parametrize("name", ["c2_twin", "c3_twin", "c4_twin", "c5_twin"])
def test_twins_run_and_rows_are_independent_units(name):
    cfg = WORKLOADS[name]
    inp = make_inputs(cfg, "cpu")
    full = orun.run(cfg, inp, ks=(1, 2))
    rows = torch.tensor([1, 0]) if cfg.block != "preln_mlp" else torch.tensor([5, 17, 199])
    part = orun.run(cfg, inp, ks=(1, 2), rows=rows)
    for l in (0, cfg.steps // 2, cfg.steps):
        sel = rows.numpy()
        np.testing.assert_allclose(part["exact"][l], full["exact"][l][sel], rtol=1e-10, atol=1e-18)
        np.testing.assert_allclose(part["hbp"][2][l], full["hbp"][2][l][sel], rtol=1e-10, atol=1e-18)
    # empirical only (not a theorem): on these small-norm blocks the error shrinks with k
    e1 = max(rel_l2(full["hbp"][1][l], full["exact"][l]) for l in range(cfg.steps + 1))
    e2 = max(rel_l2(full["hbp"][2][l], full["exact"][l]) for l in range(cfg.steps + 1))
    assert e2 <= e1
