#!/usr/bin/env python
"""Benchmark of the Highway-BP hot path: one step = one hbp_backward(k) (initial estimate, k x {all-layer
VJP, reverse scan}, parameter gradients) on a seeded synthetic workload resident in HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--k 4] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torchrun) every rank runs an independent replica of
the workload: the path has no exchange step, so there is no collective in the data path and scaling is weak.
``--impl reference`` times the fp64 CPU oracle on bounded samples of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "ms per Highway-BP backward (k iterations + parameter gradients)"
UNIT = "ms"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-detail", action="store_true", help="skip the k sweep, the other workloads and the CPU baseline")
    ap.add_argument("--others", default="c2,c3,c4",
                    help="workloads summarised under detail.other_workloads after the main one (N=1 only; '' = none)")
    return ap.parse_args()


L2_BYTES = 126e6


def config_of(w, k, touched_bytes=None):
    """touched_bytes: what one step reads and writes at least once (states, gradients, delta, the cached activations
    and scratch in the workspace); above a few L2 sizes nothing survives in L2 from one step to the next."""
    if touched_bytes is None or touched_bytes > 2 * L2_BYTES:
        l2 = "inputs_larger_than_l2 (no flush needed)"
    else:
        l2 = f"NOT larger than L2 (a step touches {touched_bytes / 1e6:.0f} MB): a latency case, not a bandwidth figure"
    return {"workload": f"{w.name}: {w.block} L={w.L} d={w.d} hidden={w.hidden} tokens={w.tokens} {w.dtype}",
            "k": k, "steps_of_scan": w.steps, "with_param_grads": True, "l2": l2, "seed": w.seed}


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per unit of work from the ncu captures summarised under
# profiles/.  An entry is used only while the kernel's sources still hash to the value recorded with the capture and
# the workload has the captured shapes; otherwise the bench line carries "traffic": null.
TRAFFIC = {
    # gemm_tc_kernel, VJP pair (dA + dY): c5_small (4 layers x 16384 tokens): 2050.448 + 1063.307 and 2531.918 + 292.011 MB;
    # c2_small (8 layers x 8192 tokens): 738.928 + 506.633 and 809.241 + 133.026 MB
    "gemm_vjp": [
        {"sources": ("gemm_tc.cu", "tc_common.cuh"), "sha256": "a0699ad7953dac89", "shape": ("preln_mlp", "bf16", 2048, 8192),
         "bytes_per_token_layer": (2050.448e6 + 1063.307e6 + 2531.918e6 + 292.011e6) / (4 * 16384),
         "profile": "profiles/gemm_tc_kernel_c5_small.md"},
        {"sources": ("gemm_tc.cu", "tc_common.cuh"), "sha256": "a0699ad7953dac89", "shape": ("preln_mlp", "bf16", 1024, 4096),
         "bytes_per_token_layer": (738.928e6 + 506.633e6 + 809.241e6 + 133.026e6) / (8 * 8192),
         "profile": "profiles/gemm_tc_kernel_c2_small.md"}],
    # scan_depth_lnstat_kernel: c5_small 605.152 MB read + 213.872 MB written for 4 steps x 16384 x 2048 elements; c2_small
    # 286.336 + 80.986 MB for 8 x 8192 x 1024 (the writes still in L2 when such a small launch ends are not in the counter)
    "scan_lnstat": [
        {"sources": ("scan.cu",), "sha256": "981b284763a28eb7", "shape": ("preln_mlp", "bf16", 2048, 8192),
         "bytes_per_state_element_step": (605.152e6 + 213.872e6) / (4 * 16384 * 2048),
         "profile": "profiles/scan_depth_lnstat_kernel_c5_small.md"},
        {"sources": ("scan.cu",), "sha256": "981b284763a28eb7", "shape": ("preln_mlp", "bf16", 1024, 4096),
         "bytes_per_state_element_step": (286.336e6 + 80.986e6) / (8 * 8192 * 1024),
         "profile": "profiles/scan_depth_lnstat_kernel_c2_small.md"}],
    # scan_ring_kernel on c3 (dram__bytes.sum.per_second x gpu__time_duration of the capture): the scan that writes the
    # next VJP's split operand 6.166 TB/s x 165.2 us, the plain one 4.769 TB/s x 101.6 us
    "scan_ring": [
        {"sources": ("scan_ring.cu", "tc_common.cuh"), "sha256": "636a8f78eb8620ef", "shape": ("rnn_tanh", "f32", 512, 0),
         "bytes_per_state_element_step": 4.769e12 * 101.6e-6 / (4096 * 32 * 512),
         "bytes_per_state_element_step_operand": 6.166e12 * 165.2e-6 / (4096 * 32 * 512),
         "profile": "profiles/scan_ring_kernel_c3.md"}],
}


def _sources_hash(names):
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2501_17086_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic(key, w):
    """Entry of TRAFFIC[key] that describes this workload's shapes, if the kernel still is the captured one, else None."""
    for t in TRAFFIC[key]:
        if (w.block, w.dtype, w.d, w.hidden) != t["shape"]:
            continue
        try:
            if _sources_hash(t["sources"]) == t["sha256"]:
                return t
        except OSError:
            pass
    return None


def algorithmic_flops(w, k):
    """VJP flops per iteration and parameter-pass flops of the MLP stacks (4dh and 6dh per token-layer)."""
    if w.block in ("mlp", "preln_mlp", "relu_mlp", "postln_mlp"):
        per = w.d * w.hidden * w.tokens * w.L
        return 4 * per, 6 * per
    if w.block == "rnn_tanh":
        rows = w.L * w.batch
        return 2 * w.d * w.d * rows, 2 * w.d * (w.d + w.in_dim) * rows
    if w.block == "gru":
        rows = w.L * w.batch
        return 6 * w.d * w.d * rows, 6 * w.d * (w.d + w.in_dim) * rows
    if w.block == "lstm":
        rows, u = w.L * w.batch, w.hidden
        return 8 * u * u * rows, 8 * u * (u + w.in_dim) * rows
    if w.block == "preln_transformer":
        n, d, s = w.tokens, w.d, w.seq
        blk = 8 * d * d * n + 5 * s * d * n + 16 * d * d * n
        wg = 8 * d * d * n + 16 * d * d * n + (2 * d * d * n + 5 * s * d * n + 4 * d * w.hidden * n)
        return blk * w.L, wg * w.L
    raise ValueError(w.block)


def forward_flops(w):
    """Flops of one forward pass (the two GEMMs of each MLP block; projections and the causal attention core of a
    decoder block; the recurrent and input products of a cell)."""
    if w.block in ("mlp", "preln_mlp", "relu_mlp", "postln_mlp"):
        return 4 * w.d * w.hidden * w.tokens * w.L
    if w.block == "preln_transformer":
        n, d, s = w.tokens, w.d, w.seq
        return (8 * d * d * n + 2 * s * d * n + 4 * d * w.hidden * n) * w.L
    rows = w.L * w.batch
    gates = {"rnn_tanh": 1, "gru": 3, "lstm": 4}[w.block]
    u = w.hidden if w.block == "lstm" else w.d
    return 2 * gates * u * (u + w.in_dim) * rows


# The paper's own timings for the recurrent experiments these shapes stand in for (Table 5 of Appendix F and the
# speed-up table of Section 5.2.2): whole TRAINING-STEP times in ms (forward + backward + update) on "A100, A40 or
# RTX A6000" GPUs with framework tensor ops, batch 128.  Context for the Highway-BP-against-BPTT ratio, not a target:
# other hardware, another quantity (a training step, not a backward pass).
PAPER_CONTEXT = {
    "g1": {"row": "1 GRU layer, L=256, 512 units", "train_step_ms": {"bp": 209, "hbp_k0": 66, "hbp_k5": 118, "hbp_k10": 166},
           "speedup_vs_bp": {"k0": 3.2, "k5": 1.8, "k10": 1.3}},
    "l1": {"row": "1 LSTM layer, L=256, 512 units", "train_step_ms": {"bp": 261, "hbp_k0": 87, "hbp_k5": 154, "hbp_k10": 218},
           "speedup_vs_bp": {"k0": 3.0, "k5": 1.7, "k10": 1.2}},
    "g2": {"row": "1 GRU layer, L=1024, 64 units", "train_step_ms": {"bp": 715, "hbp_k0": 205, "hbp_k5": 230, "hbp_k10": 248},
           "speedup_vs_bp": {"k0": 3.5, "k5": 3.1, "k10": 2.9}},
    "c3": {"row": "no row of the paper has this shape (constant gate, T=4096, batch 32); nearest in kind: 1 GRU layer, L=1024",
           "train_step_ms": {"bp": 715, "hbp_k0": 205, "hbp_k5": 230, "hbp_k10": 248},
           "speedup_vs_bp": {"k0": 3.5, "k5": 3.1, "k10": 2.9}},
}
PAPER_CONTEXT_NOTE = ("paper: training-step times (forward + backward + update), Table 5 / Section 5.2.2, on A100 / A40 / "
                      "RTX A6000 (which one per row is not stated), framework tensor ops; context, not the target")


# ----------------------------------------------------------------------------------------------- CPU oracle timing
def oracle_timing(w, k, sample, steps, warmup, max_threads=None):
    """Times the fp64 oracle's Highway-BP(k) + parameter gradients on `sample` independent units per step.
    Returns (list of seconds per step, threads used, description).  max_threads=1 limits the BLAS pools to one thread."""
    if max_threads is not None:
        from threadpoolctl import threadpool_limits
        import torch
        old = torch.get_num_threads()
        torch.set_num_threads(max_threads)
        try:
            with threadpool_limits(limits=max_threads):
                times, _, desc, scale = oracle_timing(w, k, sample, steps, warmup)
        finally:
            torch.set_num_threads(old)
        return times, max_threads, desc, scale
    import dataclasses
    import torch
    from oracle import hbp_oracle as O
    from oracle import run as orun
    from paper_2501_17086_b200.workloads import make_inputs

    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    sample, layers = sample if isinstance(sample, tuple) else (sample, None)
    # a bounded sample in depth as well where the stack is deep: the first `layers` layers (every layer costs the same),
    # so that their weights can be held in fp64 and a step times the method, not dtype conversion
    ws = dataclasses.replace(w, L=layers) if layers and layers < w.L else w
    inp = make_inputs(ws, "cpu")
    weights = ("W1", "W2", "Wq", "Wk", "Wv", "Wo", "W", "U", "a")
    if sum(t.numel() for n, t in inp.items() if n in weights) < 1.5e9:
        inp64 = {n: (t.double() if n in weights else t) for n, t in inp.items()}
    else:  # too large to hold in float64 at once: converted layer by layer inside the timed calls
        inp64 = inp
    units = {"preln_transformer": w.batch, "rnn_tanh": w.batch, "gru": w.batch, "lstm": w.batch}.get(w.block, w.tokens)
    sample = min(sample, units)
    times = []
    for it in range(warmup + steps):
        rows = torch.arange(sample) + (it * sample) % max(1, units - sample + 1)
        stack, x0, groups = orun.build_stack(ws, inp64, rows)
        xs, caches = O.forward(stack, x0)
        deltas = orun.loss_deltas(ws, xs, inp64, rows)
        t0 = time.perf_counter()
        g = O.highway_bp(stack, caches, deltas, k)
        O.param_grads(stack, caches, xs, g, groups)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    scale = (units / sample) * (w.L / ws.L)
    depth = f" and the first {ws.L} of {w.L} layers" if ws.L != w.L else ""
    desc = (f"{sample} of {units} independent units{depth} per step with the full weights, fp64 numpy; "
            f"reported value = measured time x {scale:g} (linear extrapolation)")
    return times, threads, desc, scale


def run_reference(args):
    from paper_2501_17086_b200.workloads import WORKLOADS
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOADS[args.workload]
    sample = ORACLE_SAMPLE.get(w.name, 8)
    times, threads, desc, scale = oracle_timing(w, args.k, sample, args.steps, args.warmup)
    ms_step = 1e3 * sum(times) / len(times)
    value = ms_step * scale
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(w, args.k),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in ln.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        rows = [r for t, r in self.rows if t0 <= t <= t1] or [r for _, r in self.rows[-3:]]
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------- ours
# (independent units, layers) of the oracle's bounded sample per step; layers None = the whole depth
ORACLE_SAMPLE = {"c2": 16, "c5": (4, 16), "c4": (1, 6), "c3": 2}


def measure(env, wname, k, steps, warmup, headline, detail):
    """Runs one workload: forward, warm-up, `steps` timed hbp_backward(k) calls with parameter gradients.
    headline: the full JSON line (end-to-end leg, clocks); otherwise a short summary for detail.other_workloads.
    detail: k sweep, exact BP, forward pass, graph replay, cosine with the exact gradient."""
    import torch
    from paper_2501_17086_b200 import binding, harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs

    world, local, timed = env["world"], env["local"], env["timed"]
    w = WORKLOADS[wname]
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    xin = harness.rnn_inputs(w, inp)
    x_all = ctx.forward(params, inp["x0"], xin)
    delta = harness.loss_delta(w, x_all, inp)
    grads = ctx.new_grads(with_gate=True)
    g_all = ctx.new_states()

    touched = sum(t.numel() * t.element_size() for t in (x_all, g_all, delta, ctx.workspace))
    step = lambda: ctx.backward(params, k, delta, x_all, xin, g_all=g_all, grads=grads)
    for _ in range(max(3, warmup)):
        step()
    ctx.sync_status()
    # ---- timed region: device-resident inputs
    sampler = ClockSampler(local) if headline else None
    if sampler:
        time.sleep(0.3)
    ctx.profile_enable(True)
    l0, t0 = ctx.launches, time.perf_counter()
    ms_step = timed(step, steps)
    t1 = time.perf_counter()
    launches = ctx.launches - l0
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    clocks = sampler.stop(t0, t1) if sampler else None

    # ---- end to end through the same call with host buffers: delta in from pinned memory, dL/dx_0 out.  The other
    # results (every g_l, the float parameter gradients) stay on the device, where a training step consumes them.
    e2e = None
    if headline:
        h_delta = delta.cpu().pin_memory()
        h_g0 = torch.empty_like(g_all[0], device="cpu").pin_memory()
        d_delta = torch.empty_like(delta)

        def e2e_step():
            d_delta.copy_(h_delta, non_blocking=True)
            ctx.backward(params, k, d_delta, x_all, xin, g_all=g_all, grads=grads)
            h_g0.copy_(g_all[0], non_blocking=True)

        for _ in range(2):
            e2e_step()
        e2e = {"value": timed(e2e_step, steps), "unit": UNIT, "h2d_bytes_per_step": h_delta.numel() * h_delta.element_size(),
               "d2h_bytes_per_step": h_g0.numel() * h_g0.element_size(),
               "left_on_device": "g_1..g_L and the float parameter gradients (consumed by the optimiser on the device)"}
        del h_delta, h_g0, d_delta

    # ---- roofline of the dominant kernel (the tensor-core GEMM launches of the VJP phase)
    peaks = env["peaks"]
    vjp_flops, wgrad_flops = algorithmic_flops(w, k)
    kk = min(k, w.steps)
    vjp_ms, vjp_launches = prof["vjp"]
    scan_ms, scan_launches = prof["scan"]
    wg_ms, _ = prof["wgrad"]
    es = 2 if w.dtype == "bf16" else 4
    bf16_peak = peaks.get("bf16_tflops_sustained", 1400.0)
    if w.dtype == "bf16" and vjp_ms > 0:
        achieved = vjp_flops * kk * steps / (vjp_ms * 1e-3) / 1e12
        kernel = "gemm_tc_kernel (VJP phase: dA=G*W2 with GELU' epilogue, dY=dZ*W1)"
        if w.block == "preln_transformer":
            kernel = "gemm_tc_kernel + attn_bwd kernels (whole VJP phase, algorithmic flops)"
        roofline = {"bound": "tensor", "kernel": kernel,
                    "achieved": achieved, "peak": bf16_peak, "unit": "TFLOP/s", "frac": achieved / bf16_peak,
                    "peak_source": "of measured (sustained bf16 GEMM)" if peaks else "of fallback",
                    "frac_of_burst": achieved / peaks.get("bf16_tflops", 1590.0),
                    "flops_per_launch": vjp_flops * kk * steps / max(1, vjp_launches),
                    "ms_per_launch": vjp_ms / max(1, vjp_launches), "traffic": None}
        t = measured_traffic("gemm_vjp", w)
        if t:  # bytes of one VJP pair over all layers, spread over the launches that made it
            roofline["traffic"] = t["bytes_per_token_layer"] * w.tokens * w.L * kk * steps / max(1, vjp_launches)
            roofline["traffic_source"] = t["profile"] + " (scaled by tokens x layers per launch)"
    else:
        # float data: the contraction runs on the tensor cores as three tf32 products per algorithmic product
        # (split operands), so the hardware does 3x the algorithmic flops; tf32 peak = measured bf16 peak x the
        # nominal tf32/bf16 ratio (1.1 / 2.25).  The operand split is inside the measured phase.
        alg = (vjp_flops * kk * steps / (vjp_ms * 1e-3) / 1e12) if vjp_ms else None
        # These launches are short and run at the full clock (no power cap in the clock record), so the burst figure
        # is the peak they are held to; the fraction of the sustained one is given beside it.
        tf32_peak = peaks.get("bf16_tflops", 1590.0) * 1.1 / 2.25
        tf32_sustained = bf16_peak * 1.1 / 2.25
        scan_writes_operand = w.block == "rnn_tanh" and os.environ.get("HBP_SCAN_OPERAND", "1") != "0"
        split_note = "the operand split is written by the preceding scan" if scan_writes_operand else "incl. the operand split"
        roofline = {"bound": "tensor", "kernel": f"gemm_tc_kernel, tf32 x3 (VJP phase, {split_note})",
                    "achieved": 3 * alg if alg else None, "peak": tf32_peak, "unit": "TFLOP/s (tf32, 3 per algorithmic flop)",
                    "frac": (3 * alg / tf32_peak) if alg else None, "algorithmic_tflops": alg,
                    "algorithmic_frac": (alg / tf32_peak) if alg else None,
                    "fp32_alu_peak_tflops": 148 * 128 * 2 * 1.965e9 / 1e12,
                    "frac_of_sustained": (3 * alg / tf32_sustained) if alg else None,
                    "peak_source": "of measured burst bf16 x nominal tf32/bf16 ratio" if peaks else "of fallback", "traffic": None}
    # scan: read u (+ xhat when the LayerNorm finish is fused, + the per-element gate of a GRU), write g
    tensors = 2 + (1 if w.block in ("preln_mlp", "preln_transformer", "gru", "lstm") else 0)  # per-step delta is added by the VJP GEMM epilogue
    if w.block == "postln_mlp":  # u, the non-block part c, g written; + the previous iterate when the split is shifted
        tensors = 3 + (1 if getattr(w, "gamma", 0.0) else 0)
    scan_note = None
    if w.block == "rnn_tanh" and w.dtype == "f32" and kk > 1 and os.environ.get("HBP_SCAN_OPERAND", "1") != "0":
        # every scan but the last reads u and tanh' and writes the two terms of the next VJP's operand instead of g
        tensors = (4 * (kk - 1) + 2) / kk
        scan_note = f"{kk - 1} of {kk} scans write the next VJP's split operand (4 tensors), the last writes g (2)"
    scan_bytes = tensors * w.steps * w.tokens * w.d * es
    hbm = peaks.get("hbm_gbs", 6650.0)
    scan_iter_ms = None
    if kk > 0 and scan_ms > 0:
        # the scan phase holds exactly the k scans of the iterations (g^0 is booked under "other")
        scan_iter_ms = scan_ms / steps / kk
    scan_roof = {"bound": "hbm", "kernel": "scan_depth_lnstat_kernel" if tensors >= 3 and w.loss != "every_mse" else "scan kernels",
                 "achieved": (scan_bytes / (scan_iter_ms * 1e-3) / 1e9) if scan_iter_ms else None, "peak": hbm, "unit": "GB/s",
                 "bytes_per_scan": scan_bytes, "tensors_counted": tensors, "traffic": None}
    if scan_note:
        scan_roof["note"] = scan_note
    if scan_roof["achieved"]:
        scan_roof["frac"] = scan_roof["achieved"] / hbm
    t = measured_traffic("scan_lnstat", w)
    if t:
        scan_roof["traffic"] = t["bytes_per_state_element_step"] * w.steps * w.tokens * w.d
        scan_roof["traffic_source"] = t["profile"] + " (scaled by steps)"
    t = measured_traffic("scan_ring", w)
    if t:
        scan_roof["kernel"] = "scan_ring_kernel"
        per = t["bytes_per_state_element_step"]
        if scan_note:  # the average over the phase's scans, like bytes_per_scan
            per = ((kk - 1) * t["bytes_per_state_element_step_operand"] + per) / kk
        scan_roof["traffic"] = per * w.steps * w.tokens * w.d
        scan_roof["traffic_source"] = t["profile"]

    phases = {"vjp": vjp_ms / steps, "scan": scan_ms / steps, "wgrad": wg_ms / steps}
    tflops = {"vjp": vjp_flops * kk / (vjp_ms / steps * 1e-3) / 1e12 if vjp_ms else None,
              "wgrad": wgrad_flops / (wg_ms / steps * 1e-3) / 1e12 if wg_ms else None}
    if headline:
        line = {"metric": METRIC, "value": ms_step, "unit": UNIT, "n_gpus": world, "steps": steps,
                "warmup": max(3, warmup), "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
                "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": config_of(w, k, touched),
                "working_set_gb": touched / 1e9, "clocks": clocks, "gpu_launches": launches, "e2e": e2e,
                "roofline": roofline, "scan_roofline": scan_roof, "phases_ms_per_step": phases, "tflops": tflops,
                "replicas_tokens_per_s": world * w.tokens * (w.L if w.block in ("rnn_tanh", "gru", "lstm") else 1) / (ms_step * 1e-3)}
    else:
        line = {"config": config_of(w, k, touched), "ms_per_step": ms_step, "steps": steps, "gpu_launches": launches,
                "phases_ms_per_step": phases, "tflops": tflops,
                "roofline": {x: roofline.get(x) for x in ("kernel", "achieved", "peak", "unit", "frac", "frac_of_burst", "algorithmic_frac")},
                "scan_roofline": {x: scan_roof.get(x) for x in ("kernel", "achieved", "peak", "unit", "frac", "tensors_counted")}}
    if w.name in PAPER_CONTEXT:
        line["paper_context"] = dict(PAPER_CONTEXT[w.name], note=PAPER_CONTEXT_NOTE)

    if detail:
        d = {}
        ks = (1, 2, 4, 8) if headline else ()
        for kx in ks:
            fn = lambda kx=kx: ctx.backward(params, kx, delta, x_all, xin, g_all=g_all, grads=grads)
            fn()
            d[f"hbp_k{kx}_ms"] = timed_local(torch, fn, 3)
        fn = lambda: ctx.exact(params, delta, x_all, xin, g_all=g_all, grads=grads)
        fn()
        d["exact_bp_ms"] = timed_local(torch, fn, 3)
        if w.block in ("rnn_tanh", "gru", "lstm"):
            d["hbp_over_exact_bptt"] = ms_step / d["exact_bp_ms"]
        # the forward pass (T_forward of the paper's cost model), against the same peaks
        fwd = lambda: ctx.forward(params, inp["x0"], xin, x_all=x_all)
        fwd()
        d["forward_ms"] = timed_local(torch, fwd, 3)
        ff = forward_flops(w) / (d["forward_ms"] * 1e-3) / 1e12
        d["forward_tflops"] = ff
        if w.dtype == "bf16":
            d["forward_frac"] = ff / bf16_peak
            d["forward_peak"] = "of measured (sustained bf16 GEMM)"
        else:  # the sequential recurrence is carried in double on the FP64 units
            fp64_peak = 148 * 64 * 2 * 1.965e9 / 1e12
            d["forward_frac"] = ff / fp64_peak
            d["forward_peak"] = "of the FP64 rate, 148 SMs x 64 FMA/clk x 1.965 GHz = 37.2 TFLOP/s (derived; the steps are dependent)"
        if headline:
            # the same step replayed from a CUDA graph (the calls only enqueue and never allocate): what launch overhead
            # costs on the small workloads
            try:
                graph = torch.cuda.CUDAGraph()
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph, stream=side):
                        ctx.backward(params, k, delta, x_all, xin, g_all=g_all, grads=grads)
                torch.cuda.synchronize()
                graph.replay()
                d["graph_replay_ms"] = timed_local(torch, graph.replay, 5)
                del graph
            except Exception as e:  # capture is a convenience of the host runtime: report, do not fail the bench
                d["graph_replay_ms"] = None
                d["graph_error"] = str(e)[:200]
            # Figure 5's quantity on this synthetic workload: cosine similarity of the k-iteration estimate with the
            # exact gradient, per state, computed on the device (hbp_compare); minimum and median over the states
            try:
                g_exact = ctx.exact(params, delta, x_all, xin, g_all=g_all).clone()
                cos = {}
                for kx in (1, 2, 4, 8):
                    ctx.backward(params, kx, delta, x_all, xin, g_all=g_all, grads=None)
                    s4 = binding.compare(g_all[:-1], g_exact[:-1], segments=w.steps)
                    c = s4[:, 0] / torch.sqrt(s4[:, 1] * s4[:, 2]).clamp_min(1e-300)
                    cos[f"k{kx}"] = {"min": float(c.min()), "median": float(c.median()), "last_quarter_min": float(c[3 * w.steps // 4:].min())}
                d["cosine_vs_exact"] = cos
                del g_exact
            except torch.OutOfMemoryError:
                d["cosine_vs_exact"] = None
        line["detail"] = d
    ctx.sync_status()
    ctx.close()
    del ctx, params, inp, x_all, delta, grads, g_all
    torch.cuda.empty_cache()
    return line


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2501_17086_b200.workloads import WORKLOADS

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        barrier()
        ms = torch.tensor([a.elapsed_time(b) / steps], device="cuda")
        if world > 1:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item())

    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    env = {"world": world, "local": local, "timed": timed, "peaks": peaks}
    # the k sweep and the other workloads run on one GPU only: with N > 1 every GPU is held for the timed steps alone
    want_detail = (not args.no_detail) and world == 1
    line = measure(env, args.workload, args.k, args.steps, args.warmup, headline=True, detail=want_detail)
    if want_detail:
        others = {}
        for name in [n for n in args.others.split(",") if n and n != args.workload]:
            others[name] = measure(env, name, args.k, 5, 3, headline=False, detail=True)
        if others:
            line["detail"]["other_workloads"] = others
        w = WORKLOADS[args.workload]
        sample = ORACLE_SAMPLE.get(w.name, 8)
        times, threads, desc, scale = oracle_timing(w, args.k, sample, 1, 0)
        line["cpu_baseline"] = {"value": 1e3 * times[0] * scale, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": desc, "measured_s": times[0]}
        # the same oracle held to one thread, on a quarter of the units
        s1 = (max(1, sample[0] // 4), sample[1]) if isinstance(sample, tuple) else max(1, sample // 4)
        t1, _, desc1, scale1 = oracle_timing(w, args.k, s1, 1, 0, max_threads=1)
        line["cpu_baseline"]["one_thread"] = {"value": 1e3 * t1[0] * scale1, "unit": UNIT, "cores": 1, "sample": desc1,
                                              "measured_s": t1[0]}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def timed_local(torch, fn, reps):
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
