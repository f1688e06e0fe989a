"""Glue between the synthetic workloads and the binding: parameter dicts and the loss gradient
delta_l (an INPUT of the library), formed with torch from the states the library's forward produced."""
from __future__ import annotations

import torch

from . import binding
from .workloads import Workload


def params_for(w: Workload, inputs: dict) -> dict:
    if w.block == "rnn_tanh":
        return {"W": inputs["W"], "U": inputs["U"], "a": inputs["a"]}
    if w.block in ("gru", "lstm"):
        return {"W": inputs["W"], "U": inputs["U"]}
    names = ("W1", "W2") if w.block != "preln_transformer" else ("Wq", "Wk", "Wv", "Wo", "W1", "W2")
    return {n: inputs[n] for n in names}


def rnn_inputs(w: Workload, inputs: dict):
    return inputs["X"] if w.block in ("rnn_tanh", "gru", "lstm") else None


def loss_delta(w: Workload, x_all: torch.Tensor, inputs: dict) -> torch.Tensor:
    """dLoss/dx for the workload's loss: [N, d] for a loss on the last state, [steps+1, N, d] for a loss on
    every state (entry 0 is zero)."""
    if w.loss == "final_half_sse":
        return (x_all[-1].float() - inputs["y"].float()).to(x_all.dtype)
    if w.loss == "final_mse":
        return ((x_all[-1].float() - inputs["y"].float()) * (2.0 / (w.tokens * w.d))).to(x_all.dtype)
    if w.loss == "every_mse":
        out = torch.zeros_like(x_all)
        out[1:] = ((x_all[1:].float() - inputs["Y"].float()) * (2.0 / (w.L * w.batch * w.d))).to(x_all.dtype)
        return out
    raise ValueError(w.loss)


def make_context(w: Workload) -> binding.Context:
    return binding.Context(binding.config_from_workload(w))
