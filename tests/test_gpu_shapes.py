"""Seeded random shapes through the C ABI against the oracle: widths, hidden sizes, token counts and depths that are
not multiples of any tile (only of the 16-byte vector), for every block kind and both dtypes.  Each case is small
enough for the oracle to run in full."""
import dataclasses
import random

import pytest

from oracle import run as orun
from paper_2501_17086_b200.workloads import Workload, make_inputs
from test_gpu_parity import compare, run_gpu

pytestmark = pytest.mark.gpu


def _case(seed):
    rnd = random.Random(seed)
    dtype = rnd.choice(["f32", "bf16"])
    v = 4 if dtype == "f32" else 8
    block = rnd.choice(["mlp", "preln_mlp", "rnn_tanh", "gru", "lstm", "preln_transformer"])
    if seed >= 50:   # recurrent kinds, loss on the last state only; float: with gates stored in bf16 the product of a
        # hundred of them carries sqrt(100) * 2^-9 of relative error by itself, beyond the 2e-2 bar
        block, dtype, v = ("rnn_tanh", "gru", "lstm")[seed % 3], "f32", 4
    elif seed >= 42:   # the post-LN kind, both dtypes
        block = "postln_mlp"
    elif seed >= 36:   # later seeds: the ReLU-residual kind (added after the first 36 cases were fixed)
        block, dtype, v = "relu_mlp", "f32", 4
    mult = lambda lo, hi: v * rnd.randint(max(1, lo // v), hi // v)
    if block in ("mlp", "preln_mlp", "relu_mlp", "postln_mlp"):
        return Workload(f"rand{seed}", block, dtype, L=rnd.randint(1, 6), d=mult(8, 328), hidden=mult(8, 520),
                        tokens=rnd.randint(1, 300), batch=1, seq=1, seed=5000 + seed,
                        loss=rnd.choice(["final_mse", "final_half_sse"]))
    if block == "preln_transformer":
        heads, hd = rnd.randint(1, 3), rnd.choice([32, 64]) if dtype == "f32" else 64
        batch, seq = rnd.randint(1, 3), rnd.randint(1, 210)
        return Workload(f"rand{seed}", block, dtype, L=rnd.randint(1, 2), d=heads * hd, hidden=mult(8, 260), n_heads=heads,
                        head_dim=hd, seq=seq, batch=batch, tokens=batch * seq, seed=5000 + seed)
    T, B, nin = rnd.randint(1, 150), rnd.randint(1, 40), mult(8, 40)
    loss = "final_mse" if seed >= 50 else "every_mse"   # the last seeds: recurrent kinds with a loss on the last state only
    if seed >= 50:
        T = max(T, 70)                                   # long enough for the time scans
    if block == "lstm":
        u = mult(8, 100)
        return Workload(f"rand{seed}", block, dtype, L=T, d=2 * u, hidden=u, in_dim=nin, batch=B, tokens=B,
                        seed=5000 + seed, loss=loss)
    return Workload(f"rand{seed}", block, dtype, L=T, d=mult(8, 200), in_dim=nin, batch=B, tokens=B, seed=5000 + seed,
                    loss=loss)


@pytest.mark.parametrize("seed", range(59))
def test_random_shape_matches_oracle(seed):
    w = _case(seed)
    rnd = random.Random(1000 + seed)
    ks = tuple(sorted({0, rnd.randint(1, 3), rnd.randint(1, max(1, min(w.steps, 6)))}))
    inp = make_inputs(w, "cuda")
    gpu = run_gpu(w, inp, ks)
    kmax = max(ks)
    ref = orun.run(w, inp, ks=ks, grads_for=("exact", kmax))
    compare(w, gpu, ref, ks, ("exact", kmax))
