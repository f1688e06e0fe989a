"""Edge cases of the CUDA path through the C ABI: the scan on its own against the oracle's recurrence, gated
MLP stacks (shared and per-step gates, loss on every state), degenerate sizes, and the error statuses."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import hbp_oracle as O

pytestmark = pytest.mark.gpu


def rel(a, b):
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64).reshape(b.shape) - b) / nb) if nb else float(np.linalg.norm(a))


def np64(t):
    return t.detach().float().cpu().double().numpy()


@pytest.mark.parametrize("dtype,L,rows,d,gate,every", [
    (torch.float32, 1, 1, 4, None, False),            # a single step, a single row
    (torch.float32, 7, 3, 12, "shared", True),
    (torch.float32, 300, 5, 64, "shared", True),      # time-chunked, ragged last chunk
    (torch.float32, 257, 2, 32, "per_step", True),    # time-chunked with a gate per step
    (torch.float32, 40, 700, 256, None, False),       # depth scan, many channels
    (torch.bfloat16, 33, 130, 128, "per_step", False),
    (torch.bfloat16, 200, 4, 64, "shared", True),     # time-chunked in bf16
])
def test_cumsumprod_matches_the_recurrence(dtype, L, rows, d, gate, every):
    from paper_2501_17086_b200 import binding as B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(L * 1000 + rows)
    u = torch.randn((L, rows, d), generator=gen, device="cuda").to(dtype)
    delta = torch.randn((L + 1, rows, d) if every else (rows, d), generator=gen, device="cuda").to(dtype)
    a = None
    if gate == "shared":
        a = (0.8 + 0.25 * torch.rand((d,), generator=gen, device="cuda")).to(dtype)
    elif gate == "per_step":
        a = (0.8 + 0.25 * torch.rand((L, d), generator=gen, device="cuda")).to(dtype)
    g = B.cumsumprod(u, delta, a, loss=B.LOSS_EVERY_STEP if every else B.LOSS_FINAL)
    torch.cuda.synchronize()
    # oracle: Eq. 9 solved in order on v_l = u_l + delta_l, with the carry delta_L beyond the last step
    dl = np64(delta)
    v = [np64(u[l]) + (dl[l] if every else 0.0) for l in range(L)] + [dl[L] if every else dl]
    gates = [(1.0 if a is None else np64(a if a.dim() == 1 else a[l])) for l in range(L)] + [1.0]
    ref = O.cumsumprod_sequential(v, gates)
    tol = 1e-6 if dtype == torch.float32 else 6e-3      # bf16: one rounding of the stored g_l
    for l in range(L + 1):
        assert rel(np64(g[l]), ref[l]) < tol, l


@pytest.mark.parametrize("dtype,gate", [("f32", "shared"), ("f32", "per_step"), ("bf16", "per_step")])
def test_gated_mlp_stack_with_losses_on_every_state(dtype, gate):
    from paper_2501_17086_b200 import binding as B
    L, d, h, N = 4, 64, 96, 40
    dt = torch.float32 if dtype == "f32" else torch.bfloat16
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77)
    W1 = (torch.randn((L, h, d), generator=gen, device="cuda") / d ** 0.5).to(dt)
    W2 = (torch.randn((L, d, h), generator=gen, device="cuda") / h ** 0.5 * 0.5).to(dt)
    a = (0.7 + 0.3 * torch.rand((d,) if gate == "shared" else (L, d), generator=gen, device="cuda")).to(dt)
    x0 = torch.randn((N, d), generator=gen, device="cuda").to(dt)
    delta = torch.randn((L + 1, N, d), generator=gen, device="cuda").to(dt)
    cfg = B.make_config("preln_mlp", dtype, L, d, N, hidden=h,
                        gate=B.GATE_CHANNEL_SHARED if gate == "shared" else B.GATE_CHANNEL_PER_STEP, loss=B.LOSS_EVERY_STEP)
    ctx = B.Context(cfg)
    params = {"W1": W1, "W2": W2, "a": a}
    x_all = ctx.forward(params, x0)
    got, grads = {}, {}
    for k in (0, 1, 2, 9):
        grads[k] = ctx.new_grads(with_gate=True)
        got[k] = ctx.backward(params, k, delta, x_all, grads=grads[k]).clone()
    ge = ctx.exact(params, delta, x_all)
    ctx.sync_status()
    gates = [np64(a) if gate == "shared" else np64(a[l]) for l in range(L)]
    steps = [O.MLPStep(np64(W1[l]), np64(W2[l]), True) for l in range(L)]
    stack = O.Stack(steps, gates, gate_shared=(gate == "shared"))
    xs, caches = O.forward(stack, np64(x0))
    deltas = [np64(delta[l]) for l in range(L + 1)]
    tol = 1e-5 if dtype == "f32" else 2e-2
    exact = O.exact_bp(stack, caches, deltas)
    for l in range(L + 1):
        assert rel(np64(x_all[l]), xs[l]) < tol
        assert rel(np64(ge[l]), exact[l]) < tol
    for k in (0, 1, 2, 9):
        ref = O.highway_bp(stack, caches, deltas, k)
        assert max(rel(np64(got[k][l]), ref[l]) for l in range(L + 1)) < tol, k
    ref = O.highway_bp(stack, caches, deltas, 2)
    pg = O.param_grads(stack, caches, xs, ref, [("", l) for l in range(L)])
    assert rel(np64(grads[2]["dW1"]), pg["W1"]) < tol and rel(np64(grads[2]["dW2"]), pg["W2"]) < tol
    if gate == "shared":
        assert rel(np64(grads[2]["da"]), pg["a"]) < tol
    else:
        da = np.stack([(ref[l + 1] * xs[l]).sum(axis=0) for l in range(L)])
        assert rel(np64(grads[2]["da"]), da) < tol


def test_error_statuses_on_the_device():
    from paper_2501_17086_b200 import binding as B
    cfg = B.make_config("mlp", "f32", 3, 16, 8, hidden=32)
    ctx = B.Context(cfg)
    W1 = torch.zeros((3, 32, 16), device="cuda")
    W2 = torch.zeros((3, 16, 32), device="cuda")
    params = {"W1": W1, "W2": W2}
    x0 = torch.zeros((8, 16), device="cuda")
    x_all = ctx.new_states()
    with pytest.raises(B.HbpError) as e:          # backward before any forward
        ctx.backward(params, 1, x0, x_all)
    assert e.value.code == 4
    ctx.forward(params, x0, x_all=x_all)
    with pytest.raises(B.HbpError) as e:          # negative k
        ctx.backward(params, -1, x0, x_all)
    assert e.value.code == 1
    with pytest.raises(B.HbpError) as e:          # no delta
        ctx.backward(params, 1, None, x_all)
    assert e.value.code == 1
    mis = torch.zeros(8 * 16 + 1, device="cuda")[1:].view(8, 16)   # 4-byte aligned only
    with pytest.raises(B.HbpError) as e:
        ctx.backward(params, 1, mis, x_all)
    assert e.value.code == 2
    with pytest.raises(B.HbpError) as e:          # parameter gradients asked for but a buffer is missing
        ctx.backward(params, 1, x0, x_all, grads={"dW1": torch.zeros_like(W1)})
    assert e.value.code == 1
    need = B.workspace_bytes(cfg)                 # workspace too small / misaligned
    ws = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    base = (ws.data_ptr() + 255) // 256 * 256
    h = C.c_void_p()
    assert B.lib.hbp_create(C.byref(cfg), C.c_void_p(base), need - 1, C.byref(h)) == 5
    assert B.lib.hbp_create(C.byref(cfg), C.c_void_p(base + 8), need, C.byref(h)) == 5
    ctx.sync_status()                             # the context is still usable and clean
    g = ctx.backward(params, 5, x0, x_all)        # zero weights: every g_l is delta_L (Eq. 5 with a = 1)
    torch.cuda.synchronize()
    assert torch.equal(g, x0.expand_as(g))


@pytest.mark.parametrize("name,gamma", [("c2_twin_f32", 0.2), ("c2_twin", 0.2), ("c2_twin_f32", 1.0), ("c4_twin", 0.2), ("c1", 0.5)])
def test_gamma_shifted_split_matches_oracle(name, gamma):
    """Appendix C.3, Eq. 17: K = (1 - gamma) I, each VJP gains gamma g_{l+1}; exact BP does not depend on gamma."""
    from oracle import run as orun
    from paper_2501_17086_b200 import binding as B, harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    cfg = B.config_from_workload(w)
    cfg.gamma = gamma
    ctx = B.Context(cfg)
    params = harness.params_for(w, inp)
    x_all = ctx.forward(params, inp["x0"])
    delta = harness.loss_delta(w, x_all, inp)
    ks = (0, 1, 2, w.steps)
    got = {k: ctx.backward(params, k, delta, x_all).clone() for k in ks}
    grads = ctx.new_grads()
    ctx.backward(params, 2, delta, x_all, grads=grads)
    ge = ctx.exact(params, delta, x_all)
    ctx.sync_status()
    base, x0, groups = orun.build_stack(w, inp)
    st = O.shifted_stack(base, gamma)
    xs, caches = O.forward(st, x0)
    deltas = orun.loss_deltas(w, xs, inp)
    tol = 1e-5 if w.dtype == "f32" else 2e-2
    exact = O.exact_bp(st, caches, deltas)
    shape = xs[0].shape
    for k in ks:
        ref = O.highway_bp(st, caches, deltas, k)
        worst = max(rel(np64(got[k][l]), ref[l]) for l in range(w.steps + 1))
        assert worst < tol, (k, worst)
    assert max(rel(np64(ge[l]), exact[l]) for l in range(w.steps + 1)) < tol
    pg = O.param_grads(st, caches, xs, O.highway_bp(st, caches, deltas, 2), groups)
    for n, v in pg.items():
        assert rel(np64(grads["d" + n]), v) < tol, n


@pytest.mark.parametrize("name,ks", [("gru_twin", (1, 3)), ("lstm_twin", (1, 3)), ("c3_twin", (2,)), ("c2_twin", (2,)), ("c4_twin", (2,))])
def test_cuda_core_fallback_matches_oracle(name, ks, monkeypatch):
    """HBP_FORCE_SIMT=1 (read when a context is made) keeps every GEMM and the attention backward off the
    tensor cores: the fallback kernels must meet the same bar."""
    from oracle import run as orun
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    from test_gpu_parity import compare, run_gpu
    monkeypatch.setenv("HBP_FORCE_SIMT", "1")
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    gpu = run_gpu(w, inp, ks)
    del gpu["ctx"]
    kmax = max(ks)
    ref = orun.run(w, inp, ks=ks, grads_for=("exact", kmax))
    compare(w, gpu, ref, ks, ("exact", kmax))


@pytest.mark.parametrize("mode", ["0", "1"])
@pytest.mark.parametrize("name,ks", [("c2_twin", (2,)), ("c5_twin", (3,)), ("c4_twin", (2,)), ("c3_twin", (2,)), ("gru_twin", (2,))])
def test_gemm_single_cta_and_cta_pair_modes_match_oracle(name, ks, mode, monkeypatch):
    """HBP_GEMM_PAIR (read when a context is made): 0 keeps the tensor-core GEMM on single CTAs (128 x 256 tiles),
    1 (the default) pairs CTAs (256 x 256 tiles) wherever two row blocks exist; both must meet the bar on every twin."""
    from oracle import run as orun
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    from test_gpu_parity import compare, run_gpu
    monkeypatch.setenv("HBP_GEMM_PAIR", mode)
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    gpu = run_gpu(w, inp, ks)
    del gpu["ctx"]
    kmax = max(ks)
    ref = orun.run(w, inp, ks=ks, grads_for=("exact", kmax))
    compare(w, gpu, ref, ks, ("exact", kmax))


def test_scan_with_a_status_word_reports_no_error_and_matches_the_plain_scan():
    """hbp_cumsumprod_status on the ring scan (the form with bounded waits): same result as hbp_cumsumprod, status 0."""
    from paper_2501_17086_b200 import binding as B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    L, rows, d = 700, 4, 128
    u = torch.randn((L, rows, d), generator=gen, device="cuda")
    delta = torch.randn((L + 1, rows, d), generator=gen, device="cuda")
    a = 0.9 + 0.099 * torch.rand((d,), generator=gen, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = B.cumsumprod(u, delta, a, loss=B.LOSS_EVERY_STEP, status=status)
    want = B.cumsumprod(u, delta, a, loss=B.LOSS_EVERY_STEP)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(got, want)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """The failure path of the tensor-core kernels' waits: a GEMM tile whose copy role expects bytes that nobody
    sends, every wait limited to 1 ms.  The kernel must end by itself, the status word must read HBP_ERR_TIMEOUT (8)
    once, and afterwards the same context (same tensor memory, same status word) must compute correctly."""
    import time
    from oracle import run as orun
    from paper_2501_17086_b200 import binding as B, harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = WORKLOADS["c2_twin"]
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    x_all = ctx.forward(params, inp["x0"], None)
    ctx.sync_status()
    t0 = time.perf_counter()
    ctx.selftest_wait_timeout(limit_ns=1_000_000)
    with pytest.raises(B.HbpError) as info:
        ctx.sync_status()
    assert info.value.code == 8
    assert time.perf_counter() - t0 < 5.0           # the waits gave up after milliseconds, not after their usual seconds
    ctx.sync_status()                               # reported once; the word is clean again
    # the context is usable: the same kernels, now with their copies, give the right answer
    delta = harness.loss_delta(w, x_all, inp)
    g = ctx.backward(params, 2, delta, x_all, None)
    ctx.sync_status()
    ref = orun.run(w, inp, ks=(2,))
    for l in range(w.steps + 1):
        assert rel(np64(g[l]), ref["hbp"][2][l]) < 2e-2, l


def test_kernel_modes_belong_to_the_context(monkeypatch):
    """Two contexts created under different settings keep their own modes, and a call through either launches its own
    kind of kernels however the calls are interleaved: the modes read back as created, the CUDA-core context
    reproduces its own bits after the others have run, and all agree to the bf16 tolerance."""
    from paper_2501_17086_b200 import harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = WORKLOADS["c2_twin"]
    inp = make_inputs(w, "cuda")
    monkeypatch.setenv("HBP_FORCE_SIMT", "1")
    monkeypatch.setenv("HBP_GEMM_PAIR", "0")
    simt = harness.make_context(w)
    monkeypatch.delenv("HBP_FORCE_SIMT")
    monkeypatch.delenv("HBP_GEMM_PAIR")
    pair = harness.make_context(w)               # the default: paired CTAs
    monkeypatch.setenv("HBP_GEMM_PAIR", "0")
    plain = harness.make_context(w)
    monkeypatch.delenv("HBP_GEMM_PAIR")
    assert (simt.modes & 3, pair.modes & 3, plain.modes & 3) == (1, 2, 0)
    params = harness.params_for(w, inp)
    outs = []
    for ctx in (simt, pair, plain, simt):      # interleaved: a later context's creation or use changes nothing
        x_all = ctx.forward(params, inp["x0"], None)
        delta = harness.loss_delta(w, x_all, inp)
        outs.append(ctx.backward(params, 2, delta, x_all, None).float().clone())
        ctx.sync_status()
    assert (simt.modes & 3, pair.modes & 3, plain.modes & 3) == (1, 2, 0)
    assert torch.equal(outs[0], outs[3])        # the same context computes the same bits before and after the others
    for o in outs[1:3]:
        assert float((o - outs[0]).norm() / outs[0].norm()) < 2e-2


@pytest.mark.parametrize("T,d,batch", [(200, 128, 6), (70, 256, 3), (129, 64, 5)])
def test_scan_that_writes_the_next_vjp_operand_changes_no_bit(monkeypatch, T, d, batch):
    """Float tanh RNN: between two all-step VJPs the time scan writes g_{t+1} * tanh'(z_t), split for the tensor
    cores, instead of the intermediate iterate.  It forms that product from the very float it would have stored, so
    every k gives the same bits as a context that keeps the separate pass (HBP_SCAN_OPERAND=0), parameter gradients
    included; step counts that are not a multiple of the ring's stage and a row narrower than one block included."""
    import dataclasses
    from paper_2501_17086_b200 import harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = dataclasses.replace(WORKLOADS["c3_twin"], L=T, d=d, batch=batch, tokens=batch, in_dim=32)
    inp = make_inputs(w, "cuda")
    fused = harness.make_context(w)
    monkeypatch.setenv("HBP_SCAN_OPERAND", "0")
    plain = harness.make_context(w)
    monkeypatch.delenv("HBP_SCAN_OPERAND")
    assert fused.modes & 4 and not plain.modes & 4
    params = harness.params_for(w, inp)
    X = harness.rnn_inputs(w, inp)
    for k in (1, 2, 5):
        got = []
        for ctx in (fused, plain):
            x_all = ctx.forward(params, inp["x0"], X)
            delta = harness.loss_delta(w, x_all, inp)
            grads = ctx.new_grads(with_gate=True)
            g = ctx.backward(params, k, delta, x_all, X, grads=grads)
            ctx.sync_status()
            got.append((g.clone(), {n: t.clone() for n, t in grads.items()}))
        assert torch.equal(got[0][0], got[1][0])
        for n in got[0][1]:
            assert torch.equal(got[0][1][n], got[1][1][n]), n


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_compare_matches_the_definition(dtype):
    from paper_2501_17086_b200 import binding as B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77)
    a = torch.randn((7, 33, 40), generator=gen, device="cuda").to(dtype)
    b = (a.float() + 0.1 * torch.randn((7, 33, 40), generator=gen, device="cuda")).to(dtype)
    got = B.compare(a, b, segments=7).cpu().numpy()
    again = B.compare(a, b, segments=7).cpu().numpy()
    assert (got == again).all()                       # fixed summation order
    for l in range(7):
        want = O.agreement(np64(a[l]), np64(b[l]))
        np.testing.assert_allclose(got[l], want, rtol=1e-6)   # products of floats, accumulated in double
    with pytest.raises(B.HbpError):
        B.lib.hbp_compare.restype = C.c_int
        B._check(B.lib.hbp_compare(0, 0, 10, None, None, None, None, 0, None), "hbp_compare")


@pytest.mark.parametrize("name,world,k", [("c2_twin", 2, 2), ("c2_twin", 3, 4), ("c2_twin_f32", 3, 3), ("c2_twin_f32", 5, 5),
                                          ("c4_twin", 2, 2), ("c1", 4, 3)])
def test_layer_parallel_shards_match_the_single_context_and_the_oracle(name, world, k):
    """Layer-parallel Highway-BP with all shards in this process (one GPU): contexts over layer ranges, the scan's
    carry handed over between them.  Must agree with the oracle like the single-context path does."""
    from oracle import run as orun
    from paper_2501_17086_b200 import harness, layer_parallel as LP
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    from test_gpu_parity import TOL
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    shards = [LP.Shard(w, r, world, inp) for r in range(world)]
    out = LP.run(shards, inp["x0"], k, lambda x_last: harness.loss_delta(w, x_last.unsqueeze(0), inp))
    for s in shards:
        s.ctx.sync_status()
    ref = orun.run(w, inp, ks=(k,), exact=False, grads_for=(k,))
    tol = TOL[w.dtype]
    per_step = w.steps // w.L
    for s, (g_all, grads) in zip(shards, out):
        for j in range(g_all.shape[0]):
            l = s.lo * per_step + j
            assert rel(np64(g_all[j]), ref["hbp"][k][l]) < tol, f"rank {s.rank} state {l}"
        for n, t in grads.items():
            want = ref["grads"][k][n[1:]][s.lo:s.hi]
            assert rel(np64(t), want) < tol, f"rank {s.rank} {n}"


@pytest.mark.parametrize("name,k", [("gru_twin_long", 3), ("c2_twin", 2), ("c4_twin", 2)])
def test_backward_replays_from_a_cuda_graph(name, k):
    """The calls only enqueue work on the given stream and allocate nothing, so a backward (after one eager call
    that does the one-time kernel attribute set-up) can be captured into a CUDA graph and replayed on new data in the
    same buffers: the replay must reproduce the eager result bit for bit."""
    from paper_2501_17086_b200 import harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs
    w = WORKLOADS[name]
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    xin = harness.rnn_inputs(w, inp)
    x_all = ctx.forward(params, inp["x0"], xin)
    delta = harness.loss_delta(w, x_all, inp).contiguous()
    g_all, grads = ctx.new_states(), ctx.new_grads()
    ctx.backward(params, k, delta, x_all, xin, g_all=g_all, grads=grads)       # eager: also the one-time set-up
    torch.cuda.synchronize()
    want_g, want_w = g_all.clone(), {n: t.clone() for n, t in grads.items()}
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            ctx.backward(params, k, delta, x_all, xin, g_all=g_all, grads=grads)
    g_all.zero_()
    for t in grads.values():
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ctx.sync_status()
    assert torch.equal(g_all, want_g)
    for n in grads:
        assert torch.equal(grads[n], want_w[n]), n
    delta2 = (delta.float() * 0.5).to(delta.dtype)
    want2 = ctx.backward(params, k, delta2, x_all, xin).clone()
    delta.copy_(delta2)                      # new data in the captured buffer
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(g_all, want2)
