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
