"""Seeded synthetic workloads (inputs only; none of the method's arithmetic).

The paper trains on CIFAR10, ImageNet32, Wikitext103 and MNLI (Section 5,
Table 2).  None of those is used here: every tensor below is drawn from a
seeded counter-based generator and only the *shapes and structure* of the
paper's models are kept (residual MLP stacks, a pre-LN decoder Transformer
whose layers are split into attention and feed-forward residual steps, a
gated recurrent network with a loss at every time step).

Fill order (fixed, so a seed reproduces a workload on a given device type):
one ``torch.Generator`` per workload, seeded with ``cfg.seed``; tensors are
drawn in float32 in the order listed in ``make_inputs`` and then rounded once
to the workload's dtype.  Draws made on "cuda" and on "cpu" differ; both sides
of a comparison are always fed the same realised tensors.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    block: str            # "mlp" | "preln_mlp" | "rnn_tanh" | "preln_transformer" | "gru" | "lstm" | "relu_mlp" | "postln_mlp"
    dtype: str            # "f32" | "bf16"
    L: int                # residual steps (mlp), time steps (rnn), decoder blocks (transformer)
    d: int
    hidden: int = 0
    in_dim: int = 0
    n_heads: int = 0
    head_dim: int = 0
    seq: int = 0
    batch: int = 0
    tokens: int = 0       # rows of a state: batch*seq for token models, batch for the rnn
    seed: int = 0
    loss: str = "final_mse"   # "final_half_sse" | "final_mse" | "every_mse"
    ln_eps: float = 1e-5
    gamma: float = 0.0    # shift of the residual split (post-LN workloads; Appendix C.3)
    init: str = ""        # MLP kinds: "fan_in" (variance 1/fan_in) or "small" (std 0.02, output weights 0.02/sqrt(2 steps));
                          # "" = the kind's default (fan_in for mlp / relu_mlp / postln_mlp, small for preln_mlp)

    @property
    def steps(self) -> int:
        """Residual steps seen by the scan: two per decoder block."""
        return 2 * self.L if self.block == "preln_transformer" else self.L

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


WORKLOADS = {
    # the five evaluation shapes
    "c1": Workload("c1", "mlp", "f32", L=8, d=64, hidden=256, tokens=32, seed=1001, loss="final_half_sse"),
    "c2": Workload("c2", "preln_mlp", "bf16", L=64, d=1024, hidden=4096, batch=16, seq=512, tokens=8192, seed=1002),
    "c3": Workload("c3", "rnn_tanh", "f32", L=4096, d=512, in_dim=256, batch=32, tokens=32, seed=1003, loss="every_mse"),
    # a 128-wide tanh RNN with many row tiles per SM (196608 rows): the GEMM form for products at most 128 columns
    # wide and the time scan that writes the next VJP's operand, at a size where their rings wrap many times
    "r1": Workload("r1", "rnn_tanh", "f32", L=1024, d=128, in_dim=64, batch=192, tokens=192, seed=1010, loss="every_mse"),
    "c4": Workload("c4", "preln_transformer", "bf16", L=24, d=768, hidden=3072, n_heads=12, head_dim=64,
                   seq=1024, batch=16, tokens=16384, seed=1004),
    "c5": Workload("c5", "preln_mlp", "bf16", L=128, d=2048, hidden=8192, batch=32, seq=512, tokens=16384, seed=1005),
    # GRU cells with the update gate as the residual gate, in the shapes of the paper's recurrent experiments
    # (Table of RNN hyperparameters: batch 128; 256 steps x 512 units on characters, 1024 steps x 64 units on
    # pixels); the input widths 210 and 3 are rounded up to multiples of 4 for 128-bit access
    "g1": Workload("g1", "gru", "f32", L=256, d=512, in_dim=212, batch=128, tokens=128, seed=1006, loss="every_mse"),
    "g2": Workload("g2", "gru", "f32", L=1024, d=64, in_dim=4, batch=128, tokens=128, seed=1007, loss="every_mse"),
    # LSTM in the shape of the paper's character-level experiment: 256 steps, 512 units (state [c, h] 1024 wide)
    "l1": Workload("l1", "lstm", "f32", L=256, d=1024, hidden=512, in_dim=212, batch=128, tokens=128, seed=1008, loss="every_mse"),
    # c2's shape with post-LN layers x <- LN(x + MLP(x)) (the RoBERTa-style row of Table 1)
    "p2": Workload("p2", "postln_mlp", "bf16", L=64, d=1024, hidden=4096, batch=16, seq=512, tokens=8192, seed=1009,
                   init="small", gamma=0.8),
    # c2 with 8 layers: same per-launch tile shapes, small enough for multi-pass profiler captures
    "c2_small": Workload("c2_small", "preln_mlp", "bf16", L=8, d=1024, hidden=4096, batch=16, seq=512, tokens=8192, seed=1012),
    # c5 with 4 layers: same tile shapes per launch, small enough for multi-pass profiler captures
    "c5_small": Workload("c5_small", "preln_mlp", "bf16", L=4, d=2048, hidden=8192, batch=32, seq=512, tokens=16384, seed=1015),
    # c4 with 4 decoder blocks: same per-launch shapes, small enough for multi-pass profiler captures
    "c4_small": Workload("c4_small", "preln_transformer", "bf16", L=4, d=768, hidden=3072, n_heads=12, head_dim=64,
                         seq=1024, batch=16, tokens=16384, seed=1014),
    # reduced twins: same structure, sizes the fp64 oracle runs in full; they
    # span several tiles and leave ragged tails against 128/256-wide tiles.
    "c2_twin": Workload("c2_twin", "preln_mlp", "bf16", L=5, d=256, hidden=1024, batch=1, seq=328, tokens=328, seed=2002),
    "c2_twin_f32": Workload("c2_twin_f32", "preln_mlp", "f32", L=5, d=96, hidden=200, batch=1, seq=77, tokens=77, seed=2012),
    "c3_twin": Workload("c3_twin", "rnn_tanh", "f32", L=200, d=128, in_dim=48, batch=6, tokens=6, seed=2003, loss="every_mse"),
    "gru_twin": Workload("gru_twin", "gru", "f32", L=40, d=72, in_dim=12, batch=5, tokens=5, seed=2006, loss="every_mse"),
    "gru_twin_long": Workload("gru_twin_long", "gru", "f32", L=300, d=64, in_dim=4, batch=12, tokens=12, seed=2016,
                              loss="every_mse"),
    "gru_twin_bf16": Workload("gru_twin_bf16", "gru", "bf16", L=24, d=64, in_dim=16, batch=6, tokens=6, seed=2026,
                              loss="every_mse"),
    "lstm_twin": Workload("lstm_twin", "lstm", "f32", L=40, d=72, hidden=36, in_dim=12, batch=5, tokens=5, seed=2007, loss="every_mse"),
    "lstm_twin_long": Workload("lstm_twin_long", "lstm", "f32", L=300, d=64, hidden=32, in_dim=4, batch=12, tokens=12, seed=2017,
                               loss="every_mse"),
    "lstm_twin_bf16": Workload("lstm_twin_bf16", "lstm", "bf16", L=24, d=64, hidden=32, in_dim=16, batch=6, tokens=6, seed=2027,
                               loss="every_mse"),
    "relu_twin": Workload("relu_twin", "relu_mlp", "f32", L=5, d=96, hidden=200, batch=1, seq=77, tokens=77, seed=2008),
    "postln_twin": Workload("postln_twin", "postln_mlp", "f32", L=5, d=96, hidden=200, batch=1, seq=77, tokens=77, seed=2009),
    "postln_twin_shift": Workload("postln_twin_shift", "postln_mlp", "f32", L=5, d=96, hidden=200, batch=1, seq=77, tokens=77,
                                  seed=2029, gamma=0.8),
    "postln_twin_shift_bf16": Workload("postln_twin_shift_bf16", "postln_mlp", "bf16", L=6, d=128, hidden=512, batch=1, seq=200,
                                       tokens=200, seed=2039, gamma=0.8),
    "postln_twin_bf16": Workload("postln_twin_bf16", "postln_mlp", "bf16", L=5, d=256, hidden=1024, batch=1, seq=328,
                                 tokens=328, seed=2019),
    "c4_twin": Workload("c4_twin", "preln_transformer", "bf16", L=2, d=128, hidden=512, n_heads=2, head_dim=64,
                        seq=200, batch=2, tokens=400, seed=2004),
    "c4_twin_f32": Workload("c4_twin_f32", "preln_transformer", "f32", L=2, d=64, hidden=128, n_heads=2, head_dim=32,
                            seq=50, batch=2, tokens=100, seed=2014),
    "c5_twin": Workload("c5_twin", "preln_mlp", "bf16", L=9, d=512, hidden=1536, batch=1, seq=200, tokens=200, seed=2005),
}


def _randn(gen, shape, std, device):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std


def make_inputs(cfg: Workload, device="cpu"):
    """Returns a dict of tensors in ``cfg.dtype`` on ``device``.

    Keys: mlp / preln_mlp / relu_mlp / postln_mlp: W1 [L,h,d], W2 [L,d,h], x0 [N,d], y [N,d].
    rnn_tanh: a [d], W [d,d], U [d,in], X [T,B,in], Y [T,B,d], x0 [B,d] (zeros).
    gru: W [3d,d] (variance 1/d), U [3d,in] (variance 1/in), X, Y, x0 as for rnn_tanh.
    lstm: W [4u,u] (variance 1/u), U [4u,in] (variance 1/in) with u = hidden units, d = 2u; X [T,B,in], Y [T,B,2u],
    x0 [B,2u] (zeros).
    preln_transformer: Wq, Wk, Wv, Wo [L,d,d], W1 [L,h,d], W2 [L,d,h], x0 [N,d], y [N,d].
    Standard deviations: 0.02 for Transformer-style inputs weights and
    0.02 / sqrt(2 * steps) for the weights that write into the residual stream;
    variance 1/fan_in for the plain MLP; variance 1/in_dim for U; W is 0.5 times
    an orthogonal matrix (QR of a Gaussian, signs fixed by the diagonal of R)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    dt = cfg.torch_dtype
    out = {}
    if cfg.block in ("mlp", "preln_mlp", "relu_mlp", "postln_mlp"):
        L, d, h, N = cfg.L, cfg.d, cfg.hidden, cfg.tokens
        init = cfg.init or ("small" if cfg.block == "preln_mlp" else "fan_in")
        if init == "fan_in":
            s1, s2 = 1.0 / math.sqrt(d), 1.0 / math.sqrt(h)
        else:
            s1, s2 = 0.02, 0.02 / math.sqrt(2.0 * cfg.steps)
        out["W1"] = torch.empty((L, h, d), device=dev, dtype=dt)
        out["W2"] = torch.empty((L, d, h), device=dev, dtype=dt)
        for l in range(L):  # per layer: keeps the float32 staging buffer small
            out["W1"][l] = _randn(gen, (h, d), s1, dev).to(dt)
            out["W2"][l] = _randn(gen, (d, h), s2, dev).to(dt)
        out["x0"] = _randn(gen, (N, d), 1.0, dev).to(dt)
        out["y"] = _randn(gen, (N, d), 1.0, dev).to(dt)
    elif cfg.block == "rnn_tanh":
        T, d, B, nin = cfg.L, cfg.d, cfg.batch, cfg.in_dim
        out["a"] = (0.9 + 0.099 * torch.rand((d,), generator=gen, device=dev, dtype=torch.float32)).to(dt)
        gauss = _randn(gen, (d, d), 1.0, dev).double().cpu()
        q, r = torch.linalg.qr(gauss)
        q = q * torch.sign(torch.diagonal(r)).unsqueeze(0)
        out["W"] = (0.5 * q).contiguous().to(dev).to(dt)
        out["U"] = _randn(gen, (d, nin), 1.0 / math.sqrt(nin), dev).to(dt)
        out["X"] = _randn(gen, (T, B, nin), 1.0, dev).to(dt)
        out["Y"] = _randn(gen, (T, B, d), 1.0, dev).to(dt)
        out["x0"] = torch.zeros((B, d), device=dev, dtype=dt)
    elif cfg.block == "gru":
        T, d, B, nin = cfg.L, cfg.d, cfg.batch, cfg.in_dim
        out["W"] = _randn(gen, (3 * d, d), 1.0 / math.sqrt(d), dev).to(dt)
        out["U"] = _randn(gen, (3 * d, nin), 1.0 / math.sqrt(nin), dev).to(dt)
        out["X"] = _randn(gen, (T, B, nin), 1.0, dev).to(dt)
        out["Y"] = _randn(gen, (T, B, d), 1.0, dev).to(dt)
        out["x0"] = torch.zeros((B, d), device=dev, dtype=dt)
    elif cfg.block == "lstm":
        T, d, u, B, nin = cfg.L, cfg.d, cfg.hidden, cfg.batch, cfg.in_dim
        out["W"] = _randn(gen, (4 * u, u), 1.0 / math.sqrt(u), dev).to(dt)
        out["U"] = _randn(gen, (4 * u, nin), 1.0 / math.sqrt(nin), dev).to(dt)
        out["X"] = _randn(gen, (T, B, nin), 1.0, dev).to(dt)
        out["Y"] = _randn(gen, (T, B, d), 1.0, dev).to(dt)
        out["x0"] = torch.zeros((B, d), device=dev, dtype=dt)
    elif cfg.block == "preln_transformer":
        L, d, h, N = cfg.L, cfg.d, cfg.hidden, cfg.tokens
        s_in, s_out = 0.02, 0.02 / math.sqrt(2.0 * cfg.steps)
        for name, shape, std in (("Wq", (d, d), s_in), ("Wk", (d, d), s_in), ("Wv", (d, d), s_in),
                                 ("Wo", (d, d), s_out), ("W1", (h, d), s_in), ("W2", (d, h), s_out)):
            out[name] = torch.empty((L,) + shape, device=dev, dtype=dt)
        for l in range(L):
            for name, std in (("Wq", s_in), ("Wk", s_in), ("Wv", s_in), ("Wo", s_out), ("W1", s_in), ("W2", s_out)):
                out[name][l] = _randn(gen, tuple(out[name].shape[1:]), std, dev).to(dt)
        out["x0"] = _randn(gen, (N, d), 1.0, dev).to(dt)
        out["y"] = _randn(gen, (N, d), 1.0, dev).to(dt)
    else:
        raise ValueError(f"unknown block kind {cfg.block!r}")
    if "Y" in out:
        out["y"] = out["Y"][-1]  # target of the last state, for recurrent workloads with a loss on the last state only
    return out
