"""The N > 1 path on CPU (gloo, world size 2): ranks work on disjoint sets of independent units, need no
exchange for the state gradients, and a data-parallel job would add exactly one sum of the parameter
gradients; the benchmark's timing reduction is a max over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import run as orun
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = WORKLOADS["c2_twin_f32"]
    inp = make_inputs(w, "cpu")                      # same seed on every rank: replicated weights
    rows = torch.arange(rank, w.tokens, world)       # this rank's shard of tokens
    res = orun.run(w, inp, ks=(2,), rows=rows, grads_for=(2,))
    grads = {n: torch.from_numpy(v.copy()) for n, v in res["grads"][2].items()}
    for t in grads.values():
        dist.all_reduce(t, op=dist.ReduceOp.SUM)     # the one collective of a data-parallel job
    ms = torch.tensor([10.0 + rank])
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)        # bench.py's timing reduction
    if rank == 0:
        full = orun.run(w, inp, ks=(2,), grads_for=(2,))
        ok = all(np.allclose(grads[n].numpy(), full["grads"][2][n], rtol=1e-9, atol=1e-15) for n in grads)
        sel = rows.numpy()
        ok = ok and np.allclose(res["hbp"][2][0], full["hbp"][2][0][sel], rtol=1e-10, atol=1e-18)
        out.put((ok, float(ms.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_units_and_sum_parameter_gradients():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok, ms = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok and ms == 11.0


class _OracleShard:
    """Stands in for layer_parallel.Shard on a machine without a GPU: the same interface, the local arithmetic done
    by the fp64 oracle, so that the orchestration (pipeline, all-gather, carries) is what this test exercises."""

    def __init__(self, w, rank, world, inp):
        from oracle import hbp_oracle as O
        from paper_2501_17086_b200.layer_parallel import layer_range
        self.O, self.w, self.rank, self.world = O, w, rank, world
        self.lo, self.hi = layer_range(w.L, rank, world)
        self.stack = O.mlp_stack([t.double().numpy() for t in inp["W1"][self.lo:self.hi]],
                                 [t.double().numpy() for t in inp["W2"][self.lo:self.hi]], True, w.ln_eps)
        self.last = rank == world - 1

    def forward(self, x_in):
        self.xs, self.caches = self.O.forward(self.stack, x_in.double().numpy())
        return torch.from_numpy(self.xs[-1])

    def start(self, delta_last):
        n = len(self.xs)
        self.delta = delta_last.double().numpy() if self.last else np.zeros_like(self.xs[0])
        self.g = [self.delta.copy() for _ in range(n)]
        return torch.from_numpy(self.g[0])

    def iterate(self):
        L = len(self.g) - 1
        u = [self.stack.steps[l].vjp(self.caches[l], self.g[l + 1]) for l in range(L)]
        new = [None] * (L + 1)
        new[L] = self.delta.copy()
        for l in range(L - 1, -1, -1):
            new[l] = new[l + 1] + u[l]
        self.g = new
        return torch.from_numpy(self.g[0])

    def apply_carry(self, carry):
        self.g = [g + carry.numpy() for g in self.g]

    def param_grads(self):
        return None

    @property
    def g_all(self):
        return self.g


def _lp_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import dataclasses
    from oracle import hbp_oracle as O
    from oracle import run as orun
    from paper_2501_17086_b200 import layer_parallel as LP
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = dataclasses.replace(WORKLOADS["c2_twin_f32"], tokens=9, seq=9)
    inp = make_inputs(w, "cpu")
    shard = _OracleShard(w, rank, world, inp)

    def carries(firsts):   # the same reverse cumulative sum over ranks, by the oracle's scan
        g = O.cumsumprod_sequential([f.numpy() for f in firsts], [1.0] * len(firsts))
        return [torch.from_numpy(x) for x in g] + [torch.zeros_like(firsts[0])]

    loss = lambda x_last: (x_last - inp["y"].double()) * (2.0 / (w.tokens * w.d))
    (g_local, _), = LP.run([shard], inp["x0"].double(), 3, loss, exchange=LP.dist_exchange, pipe=LP.dist_pipe, carries=carries)
    ref = orun.run(w, inp, ks=(3,), exact=False)
    ok = all(np.allclose(g_local[j], ref["hbp"][3][shard.lo + j], rtol=1e-10, atol=1e-16) for j in range(len(g_local)))
    flag = torch.tensor([1.0 if ok else 0.0])
    dist.all_reduce(flag, op=dist.ReduceOp.MIN)
    if rank == 0:
        out.put(bool(flag.item() == 1.0))
    dist.barrier()
    dist.destroy_process_group()


def test_layer_parallel_orchestration_on_two_ranks():
    """Pipeline forward, one all-gather per iteration and the carries, with one shard per gloo rank; the local
    arithmetic is the oracle's, the result must be Highway-BP(3) of the whole stack."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_lp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ok = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok


def test_layer_ranges_partition_the_stack():
    from paper_2501_17086_b200.layer_parallel import layer_range
    for L in (1, 5, 24, 64):
        for world in (1, 2, 3, 5, 8):
            if world > L:
                continue
            r = [layer_range(L, k, world) for k in range(world)]
            assert r[0][0] == 0 and r[-1][1] == L
            assert all(r[i][1] == r[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in r]
            assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
