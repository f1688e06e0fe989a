"""Drives the fp64 oracle on a synthetic workload (TEST INFRASTRUCTURE ONLY).

Turns a workload description and its realised input tensors into an oracle
``Stack``, forms the loss gradients delta_l from the oracle's OWN forward pass,
and runs exact BP / Highway-BP / the parameter-gradient pass.  Nothing here is
used by the CUDA library.

Independent units.  Every block acts on tokens (MLP stacks), sequences
(Transformer) or batch rows (RNN) independently, so running the oracle on a
subset of units with the full weights gives exactly those rows of every state
gradient.  ``rows`` selects such a subset; the loss normalisation still uses
the size of the full problem.
"""
from __future__ import annotations

import time

import numpy as np

from . import hbp_oracle as O


class F64Items:
    """container[i] -> float64 numpy array, for torch tensors of any dtype."""

    def __init__(self, t):
        self.t = t

    def __len__(self):
        return self.t.shape[0]

    def __getitem__(self, i):
        return self.t[i].detach().to("cpu").double().numpy()


def _np(t):
    return t.detach().to("cpu").double().numpy()


def build_stack(cfg, inputs, rows=None):
    """Returns (stack, x0, groups) for the oracle; ``rows`` = sampled unit indices."""
    if cfg.block in ("mlp", "preln_mlp"):
        stack = O.mlp_stack(F64Items(inputs["W1"]), F64Items(inputs["W2"]), cfg.block == "preln_mlp", cfg.ln_eps)
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", l) for l in range(cfg.L)]
    elif cfg.block == "relu_mlp":
        stack = O.relu_mlp_stack(F64Items(inputs["W1"]), F64Items(inputs["W2"]))
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", l) for l in range(cfg.L)]
    elif cfg.block == "postln_mlp":
        stack = O.postln_mlp_stack(F64Items(inputs["W1"]), F64Items(inputs["W2"]), cfg.ln_eps, cfg.gamma)
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", l) for l in range(cfg.L)]
    elif cfg.block == "rnn_tanh":
        X = inputs["X"] if rows is None else inputs["X"][:, rows]
        stack = O.rnn_stack(_np(inputs["W"]), _np(inputs["U"]), _np(inputs["a"]), F64Items(X))
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", None)] * cfg.L
    elif cfg.block == "gru":
        X = inputs["X"] if rows is None else inputs["X"][:, rows]
        stack = O.gru_stack(_np(inputs["W"]), _np(inputs["U"]), F64Items(X))
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", None)] * cfg.L
    elif cfg.block == "lstm":
        X = inputs["X"] if rows is None else inputs["X"][:, rows]
        stack = O.lstm_stack(_np(inputs["W"]), _np(inputs["U"]), F64Items(X))
        x0 = _np(inputs["x0"] if rows is None else inputs["x0"][rows])
        groups = [("", None)] * cfg.L
    elif cfg.block == "preln_transformer":
        stack = O.transformer_stack(*(F64Items(inputs[n]) for n in ("Wq", "Wk", "Wv", "Wo", "W1", "W2")),
                                    cfg.n_heads, cfg.ln_eps)
        x0 = inputs["x0"].reshape(cfg.batch, cfg.seq, cfg.d)
        x0 = _np(x0 if rows is None else x0[rows])
        groups = [("", l // 2) for l in range(2 * cfg.L)]
    else:
        raise ValueError(cfg.block)
    return stack, x0, groups


def loss_deltas(cfg, xs, inputs, rows=None):
    """delta_l = dL_l/dx_l for the workload's loss, from the oracle's states."""
    L = len(xs) - 1
    deltas = [np.zeros_like(xs[0]) for _ in range(L + 1)]
    if cfg.loss in ("final_half_sse", "final_mse"):
        y = inputs["y"]
        if cfg.block == "preln_transformer":
            y = y.reshape(cfg.batch, cfg.seq, cfg.d)
        y = _np(y if rows is None else y[rows])
        scale = 1.0 if cfg.loss == "final_half_sse" else 2.0 / float(cfg.tokens * cfg.d)
        deltas[L] = scale * (xs[L] - y)
    elif cfg.loss == "every_mse":
        Y = inputs["Y"] if rows is None else inputs["Y"][:, rows]
        scale = 2.0 / float(cfg.L * cfg.batch * cfg.d)
        for t in range(1, L + 1):
            deltas[t] = scale * (xs[t] - _np(Y[t - 1]))
    else:
        raise ValueError(cfg.loss)
    return deltas


def run(cfg, inputs, ks=(), rows=None, exact=True, grads_for=(), timing=None):
    """Forward, then exact BP and Highway-BP for each k in ``ks``.

    Returns a dict with "xs", "deltas", "exact" (list of g_l), "hbp" {k: list},
    "grads" {"exact" or k: dict} for the entries of ``grads_for``."""
    t0 = time.perf_counter()
    stack, x0, groups = build_stack(cfg, inputs, rows)
    xs, caches = O.forward(stack, x0)
    deltas = loss_deltas(cfg, xs, inputs, rows)
    t1 = time.perf_counter()
    out = dict(xs=xs, deltas=deltas, hbp={}, grads={}, stack=stack, caches=caches, groups=groups)
    if exact:
        out["exact"] = O.exact_bp(stack, caches, deltas)
        if "exact" in grads_for:
            out["grads"]["exact"] = O.param_grads(stack, caches, xs, out["exact"], groups)
    t2 = time.perf_counter()
    # one run to the largest k: iterate j of that run IS Highway-BP with k = j (each iteration starts from the previous one)
    history = O.highway_bp(stack, caches, deltas, max(ks), return_all=True) if ks else []
    for k in ks:
        out["hbp"][k] = history[k]
        if k in grads_for:
            out["grads"][k] = O.param_grads(stack, caches, xs, out["hbp"][k], groups)
    t3 = time.perf_counter()
    if timing is not None:
        timing.update(forward_s=t1 - t0, exact_s=t2 - t1, hbp_s=t3 - t2)
    return out
