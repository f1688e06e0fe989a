"""Layer-parallel Highway-BP (the multi-device setting of the paper's discussion: every device holds a contiguous
range of layers; all block VJPs of an iteration run at the same time on all devices, and only the scan along the
residual path crosses devices).

Plumbing only: which layers a rank holds, what it sends to whom, and the order of the calls.  Every arithmetic step is
a call into the C ABI on the rank's own context (`hbp_forward`, `hbp_iterate`, `hbp_add_carry`, `hbp_param_grads`).

With residual gates equal to one, state l depends on the scan's carry-in with coefficient one, so the scan over all
devices is: each rank scans its layers from a zero carry, the ranks exchange the value each scan reached at its
first layer (one [N, d] tensor per rank: an all-gather), and every rank adds the sum over the ranks behind it to all
of its states.  That sum is also the new value at the rank's upper boundary, which the next iteration's VJP of the
rank's last layer needs, so one all-gather per iteration is the whole exchange.  The forward pass is the usual
pipeline: a rank receives the state at its lower boundary, runs its layers and passes the last state on.

`Shard` is one rank's part; `run` drives any number of shards through the phases with an `exchange` callable, so the
same code serves one shard per process with `torch.distributed` (`dist_exchange`) and several shards in one process
(`local_exchange`), which is how a single GPU checks the scheme.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding, harness
from .workloads import Workload

_PER_LAYER = ("W1", "W2", "Wq", "Wk", "Wv", "Wo")


def layer_range(L: int, rank: int, world: int):
    """Contiguous, as even as possible: the first L % world ranks hold one layer more."""
    base, extra = divmod(L, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def carries_over_ranks(firsts):
    """carry[r] = sum over the ranks behind r (holding later layers) of what their scans reached at their first
    layer: itself a reverse CumSumProd with unit gates over the rank axis (the gather-scan-scatter form of the
    distributed scan), computed by the library's scan.  Returns [world + 1, N, d]; rank r's carry is entry r + 1 and
    the last entry (the last rank's carry) is zero."""
    u = torch.stack(list(firsts))
    return binding.cumsumprod(u, torch.zeros_like(u[0]))


class Shard:
    def __init__(self, w: Workload, rank: int, world: int, inputs: dict):
        if w.block not in ("mlp", "preln_mlp", "preln_transformer") or w.loss == "every_mse":
            raise ValueError("layer-parallel runs need gates equal to one and a loss on the last state")
        if world > w.L:
            raise ValueError("more ranks than layers")
        self.w, self.rank, self.world = w, rank, world
        self.lo, self.hi = layer_range(w.L, rank, world)
        self.local = dataclasses.replace(w, L=self.hi - self.lo, name=f"{w.name}[{self.lo}:{self.hi}]")
        self.ctx = harness.make_context(self.local)
        self.params = {n: inputs[n][self.lo:self.hi] for n in _PER_LAYER if n in inputs}
        self.x_all = self.g_all = None
        self.zero = torch.zeros((w.tokens, w.d), dtype=w.torch_dtype, device="cuda")

    @property
    def last(self) -> bool:
        return self.rank == self.world - 1

    def forward(self, x_in):
        self.x_all = self.ctx.forward(self.params, x_in, None, x_all=self.x_all)
        return self.x_all[-1]

    def start(self, delta_last):
        """g^0 from a zero carry: all zeros, except on the last rank where every state is delta_L."""
        self.delta = delta_last if self.last else self.zero
        if self.g_all is None:
            self.g_all = self.ctx.new_states()
        self.g_all.zero_()  # memory initialisation; the values are produced by add_carry below
        if self.last:
            self.ctx.add_carry(self.delta, self.g_all)
        return self.g_all[0]

    def iterate(self):
        """All local VJPs from the current iterate, then the local scan from a zero carry (delta_L on the last rank)."""
        self.ctx.iterate(self.params, self.delta, self.x_all, self.g_all)
        return self.g_all[0]

    def apply_carry(self, carry):
        if carry is not None:
            self.ctx.add_carry(carry, self.g_all)

    def param_grads(self):
        grads = self.ctx.new_grads()
        return self.ctx.param_grads(self.params, self.x_all, self.g_all, grads)


def local_exchange(firsts):
    """Several shards in one process: everything is already here."""
    return list(firsts)


def dist_exchange(firsts):
    """One shard per process: all-gather of the [N, d] tensor each rank's scan reached at its first layer."""
    import torch.distributed as dist
    (mine,) = firsts
    out = [torch.empty_like(mine) for _ in range(dist.get_world_size())]
    dist.all_gather(out, mine.contiguous())
    return out


def dist_pipe(x, src, dst):
    """Moves a boundary state from rank src to rank dst (one shard per process): the sender passes x, the receiver
    passes a tensor of the right shape to fill and gets it back."""
    import torch.distributed as dist
    if dist.get_rank() == src:
        dist.send(x.contiguous(), dst)
        return x
    dist.recv(x, src)
    return x


def run(shards, x0, k, loss_delta, exchange=local_exchange, pipe=None, carries=carries_over_ranks):
    """Forward through the pipeline, then Highway-BP(k) and the parameter gradients.  `shards` are this process's
    shards in rank order (all of them, or one); `loss_delta(x_last)` gives delta_L on the rank that holds the last
    layer; `pipe(x, src, dst)` moves a boundary state between processes (None when all shards are local);
    `carries` turns the gathered first-layer values into the per-rank carries.
    Returns the per-shard (g_all, grads)."""
    x = x0
    for s in shards:
        if pipe is not None and s.rank > 0:
            x = pipe(torch.empty_like(x0), s.rank - 1, s.rank)
        x = s.forward(x)
        if pipe is not None and not s.last:
            pipe(x, s.rank, s.rank + 1)
    delta_last = loss_delta(x) if shards[-1].last else None

    def scan_step(firsts):
        carry = carries(exchange(firsts))
        for s in shards:
            if not s.last:
                s.apply_carry(carry[s.rank + 1])

    scan_step([s.start(delta_last).clone() for s in shards])
    for _ in range(min(k, shards[0].w.steps)):
        scan_step([s.iterate().clone() for s in shards])
    return [(s.g_all, s.param_grads()) for s in shards]
