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
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-detail", action="store_true", help="skip the k sweep and the CPU baseline")
    return ap.parse_args()


def config_of(w, k):
    return {"workload": f"{w.name}: {w.block} L={w.L} d={w.d} hidden={w.hidden} tokens={w.tokens} {w.dtype}",
            "k": k, "steps_of_scan": w.steps, "with_param_grads": True,
            "l2": "inputs_larger_than_l2 (no flush needed)", "seed": w.seed}


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per unit of work from the ncu captures summarised under
# profiles/.  An entry is used only while the kernel's sources still hash to the value recorded with the capture and
# the workload has the captured shapes; otherwise the bench line carries "traffic": null.
TRAFFIC = {
    # gemm_tc_kernel, VJP pair (dA + dY) on c2_small: 1242.949 MB + 895.901 MB for 8 layers x 8192 tokens
    "gemm_vjp": {"sources": ("gemm_tc.cu", "tc_common.cuh"),
                 "sha256": "79b4e446ad5f9877",
                 "shape": ("preln_mlp", "bf16", 1024, 4096), "bytes_per_token_layer": (1242.949e6 + 895.901e6) / (8 * 8192),
                 "profile": "profiles/gemm_tc_kernel_c2_small.md"},
    # scan_depth_lnstat_kernel on c2_small: 286.271 MB read + 80.401 MB written for 8 steps x 8192 x 1024 elements
    # (the writes still in L2 when that small launch ends are not in the counter)
    "scan_lnstat": {"sources": ("scan.cu",), "sha256": "5efee60609bc121d", "shape": ("preln_mlp", "bf16", 1024, 4096),
                    "bytes_per_state_element_step": (286.271e6 + 80.401e6) / (8 * 8192 * 1024),
                    "profile": "profiles/scan_depth_lnstat_kernel_c2_small.md"},
    # scan_ring_kernel on c3: 268.520 MB read + 217.638 MB written per scan
    "scan_ring": {"sources": ("scan_ring.cu", "tc_common.cuh"), "sha256": "edb684e7b31e74f9", "shape": ("rnn_tanh", "f32", 512, 0),
                  "bytes_per_state_element_step": (268.520e6 + 217.638e6) / (4096 * 32 * 512),
                  "profile": "profiles/scan_ring_kernel_c3.md"},
}


def _sources_hash(names):
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2501_17086_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic(key, w):
    """Entry of TRAFFIC if it still describes the built kernel and this workload's shapes, else None."""
    t = TRAFFIC[key]
    if (w.block, w.dtype, w.d, w.hidden) != t["shape"]:
        return None
    try:
        if _sources_hash(t["sources"]) != t["sha256"]:
            return None
    except OSError:
        return None
    return t


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


# ----------------------------------------------------------------------------------------------- CPU oracle timing
def oracle_timing(w, k, sample, steps, warmup):
    """Times the fp64 oracle's Highway-BP(k) + parameter gradients on `sample` independent units per step.
    Returns (list of seconds per step, threads used, description)."""
    import numpy as np
    import torch
    from oracle import hbp_oracle as O
    from oracle import run as orun
    from paper_2501_17086_b200.workloads import make_inputs

    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    inp = make_inputs(w, "cpu")
    # full float64 copies of the weights once, so that a step times the method and not dtype conversion
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
        stack, x0, groups = orun.build_stack(w, inp64, rows)
        xs, caches = O.forward(stack, x0)
        deltas = orun.loss_deltas(w, xs, inp64, rows)
        t0 = time.perf_counter()
        g = O.highway_bp(stack, caches, deltas, k)
        O.param_grads(stack, caches, xs, g, groups)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    desc = (f"{sample} of {units} independent units per step with the full weights, fp64 numpy; "
            f"reported value = measured time x {units}/{sample} (linear extrapolation)")
    return times, threads, desc, units / sample


def run_reference(args):
    from paper_2501_17086_b200.workloads import WORKLOADS
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOADS[args.workload]
    sample = {"c2": 16, "c5": 4, "c4": 1, "c3": 2}.get(w.name, 8)
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
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2501_17086_b200 import binding, harness
    from paper_2501_17086_b200.workloads import WORKLOADS, make_inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    w = WORKLOADS[args.workload]
    k = args.k
    inp = make_inputs(w, "cuda")
    ctx = harness.make_context(w)
    params = harness.params_for(w, inp)
    xin = harness.rnn_inputs(w, inp)
    x_all = ctx.forward(params, inp["x0"], xin)
    delta = harness.loss_delta(w, x_all, inp)
    grads = ctx.new_grads(with_gate=True)
    g_all = ctx.new_states()

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

    step = lambda: ctx.backward(params, k, delta, x_all, xin, g_all=g_all, grads=grads)
    for _ in range(max(3, args.warmup)):
        step()
    ctx.sync_status()
    # ---- timed region: device-resident inputs
    sampler = ClockSampler(local)
    time.sleep(0.3)
    ctx.profile_enable(True)
    l0, t0 = ctx.launches, time.perf_counter()
    ms_step = timed(step, args.steps)
    t1 = time.perf_counter()
    launches = ctx.launches - l0
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    clocks = sampler.stop(t0, t1)

    # ---- end to end through the same call with host buffers: delta in from pinned memory, dL/dx_0 out
    h_delta = delta.cpu().pin_memory()
    h_g0 = torch.empty_like(g_all[0], device="cpu").pin_memory()
    d_delta = torch.empty_like(delta)

    def e2e_step():
        d_delta.copy_(h_delta, non_blocking=True)
        ctx.backward(params, k, d_delta, x_all, xin, g_all=g_all, grads=grads)
        h_g0.copy_(g_all[0], non_blocking=True)

    for _ in range(2):
        e2e_step()
    e2e_ms = timed(e2e_step, args.steps)

    # ---- roofline of the dominant kernel (the tensor-core GEMM launches of the VJP phase)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    vjp_flops, wgrad_flops = algorithmic_flops(w, k)
    kk = min(k, w.steps)
    vjp_ms, vjp_launches = prof["vjp"]
    scan_ms, scan_launches = prof["scan"]
    wg_ms, _ = prof["wgrad"]
    es = 2 if w.dtype == "bf16" else 4
    if w.dtype == "bf16" and vjp_ms > 0:
        peak = peaks.get("bf16_tflops_sustained", 1400.0)
        achieved = vjp_flops * kk * args.steps / (vjp_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel (VJP phase: dA=G*W2 with GELU' epilogue, dY=dZ*W1)",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_source": "of measured (sustained bf16 GEMM)" if peaks else "of fallback",
                    "frac_of_burst": achieved / peaks.get("bf16_tflops", 1590.0),
                    "flops_per_launch": vjp_flops * kk * args.steps / max(1, vjp_launches),
                    "ms_per_launch": vjp_ms / max(1, vjp_launches), "traffic": None}
        t = measured_traffic("gemm_vjp", w)
        if t:  # bytes of one VJP pair over all layers, spread over the launches that made it
            roofline["traffic"] = t["bytes_per_token_layer"] * w.tokens * w.L * kk * args.steps / max(1, vjp_launches)
            roofline["traffic_source"] = t["profile"] + " (scaled by tokens x layers per launch)"
    else:
        # float data: the contraction runs on the tensor cores as three tf32 products per algorithmic product
        # (split operands), so the hardware does 3x the algorithmic flops; tf32 peak = measured bf16 peak x the
        # nominal tf32/bf16 ratio (1.1 / 2.25).  The split pre-pass is inside the measured phase.
        alg = (vjp_flops * kk * args.steps / (vjp_ms * 1e-3) / 1e12) if vjp_ms else None
        bf16_peak = peaks.get("bf16_tflops_sustained", 1400.0)
        tf32_peak = bf16_peak * 1.1 / 2.25
        roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel, tf32 x3 (VJP phase, incl. the operand split pre-pass)",
                    "achieved": 3 * alg if alg else None, "peak": tf32_peak, "unit": "TFLOP/s (tf32, 3 per algorithmic flop)",
                    "frac": (3 * alg / tf32_peak) if alg else None, "algorithmic_tflops": alg,
                    "fp32_alu_peak_tflops": 148 * 128 * 2 * 1.965e9 / 1e12,
                    "peak_source": "of measured bf16 x nominal tf32/bf16 ratio" if peaks else "of fallback", "traffic": None}
    # scan: read u (+ xhat when the LayerNorm finish is fused, + the per-element gate of a GRU), write g
    tensors = 2 + (1 if w.block in ("preln_mlp", "preln_transformer", "gru", "lstm") else 0)  # per-step delta is added by the VJP GEMM epilogue
    if w.block == "postln_mlp":  # u, the non-block part c, g written; + the previous iterate when the split is shifted
        tensors = 3 + (1 if getattr(w, "gamma", 0.0) else 0)
    scan_bytes = tensors * w.steps * w.tokens * w.d * es
    hbm = peaks.get("hbm_gbs", 6650.0)
    scan_iter_ms = None
    if kk > 0 and scan_ms > 0:
        # the scan phase holds exactly the k scans of the iterations (g^0 is booked under "other")
        scan_iter_ms = scan_ms / args.steps / kk
    scan_roof = {"bound": "hbm", "kernel": "scan_depth_lnstat_kernel" if tensors >= 3 and w.loss != "every_mse" else "scan kernels",
                 "achieved": (scan_bytes / (scan_iter_ms * 1e-3) / 1e9) if scan_iter_ms else None, "peak": hbm, "unit": "GB/s",
                 "bytes_per_scan": scan_bytes, "tensors_counted": tensors, "traffic": None}
    if scan_roof["achieved"]:
        scan_roof["frac"] = scan_roof["achieved"] / hbm
    t = measured_traffic("scan_lnstat", w)
    if t:
        scan_roof["traffic"] = t["bytes_per_state_element_step"] * w.steps * w.tokens * w.d
        scan_roof["traffic_source"] = t["profile"] + " (scaled by steps)"
    t = measured_traffic("scan_ring", w)
    if t:
        scan_roof["kernel"] = "scan_ring_kernel"
        scan_roof["traffic"] = t["bytes_per_state_element_step"] * w.steps * w.tokens * w.d
        scan_roof["traffic_source"] = t["profile"]

    line = {"metric": METRIC, "value": ms_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": config_of(w, k),
            "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_ms, "unit": UNIT, "h2d_bytes_per_step": h_delta.numel() * h_delta.element_size(),
                    "d2h_bytes_per_step": h_g0.numel() * h_g0.element_size()},
            "roofline": roofline, "scan_roofline": scan_roof,
            "phases_ms_per_step": {"vjp": vjp_ms / args.steps, "scan": scan_ms / args.steps, "wgrad": wg_ms / args.steps},
            "tflops": {"vjp": vjp_flops * kk / (vjp_ms / args.steps * 1e-3) / 1e12 if vjp_ms else None,
                       "wgrad": wgrad_flops / (wg_ms / args.steps * 1e-3) / 1e12 if wg_ms else None},
            "replicas_tokens_per_s": world * w.tokens * (w.L if w.block in ("rnn_tanh", "gru", "lstm") else 1) / (ms_step * 1e-3)}

    if not args.no_detail and rank == 0:
        detail = {}
        for kx in (1, 2, 4, 8):
            fn = lambda kx=kx: ctx.backward(params, kx, delta, x_all, xin, g_all=g_all, grads=grads)
            fn()
            detail[f"hbp_k{kx}_ms"] = timed_local(torch, fn, 3)
        fn = lambda: ctx.exact(params, delta, x_all, xin, g_all=g_all, grads=grads)
        fn()
        detail["exact_bp_ms"] = timed_local(torch, fn, 3)
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
            detail["graph_replay_ms"] = timed_local(torch, graph.replay, 5)
            del graph
        except Exception as e:  # capture is a convenience of the host runtime: report, do not fail the bench
            detail["graph_replay_ms"] = None
            detail["graph_error"] = str(e)[:200]
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
            detail["cosine_vs_exact"] = cos
            del g_exact
        except torch.OutOfMemoryError:
            detail["cosine_vs_exact"] = None
        line["detail"] = detail
        if world == 1:
            sample = {"c2": 16, "c5": 4, "c4": 1, "c3": 2}.get(w.name, 8)
            times, threads, desc, scale = oracle_timing(w, k, sample, 1, 0)
            line["cpu_baseline"] = {"value": 1e3 * times[0] * scale, "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "sample": desc, "measured_s": times[0]}
    ctx.sync_status()
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
