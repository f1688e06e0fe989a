"""Host logic of bench.py that needs no GPU: the flop accounting behind the roofline fractions, the table of
profiled DRAM traffic (an entry may only be used while the kernel sources are the profiled ones), and the JSON line of
the reference arm (the oracle timed on the host cores)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2501_17086_b200.workloads import WORKLOADS  # noqa: E402


def test_flops_of_the_named_configurations():
    """One Highway-BP iteration costs two GEMMs per MLP block (4 d h flops per token and layer), the parameter pass
    three (6 d h); a recurrent cell 2 d^2 per row and step; a decoder block its projections (8 d^2), the five causal
    block products of the attention backward (5 S d) and the MLP (16 d^2 with h = 4 d)."""
    vjp, wg = bench.algorithmic_flops(WORKLOADS["c2"], 4)
    assert vjp == 4 * 1024 * 4096 * 8192 * 64 and wg == 6 * 1024 * 4096 * 8192 * 64
    assert abs(vjp / 8.796e12 - 1) < 1e-3
    vjp, wg = bench.algorithmic_flops(WORKLOADS["c5"], 4)
    assert abs(vjp / 140.7e12 - 1) < 1e-3 and abs(wg / 211.1e12 - 1) < 1e-3
    vjp, wg = bench.algorithmic_flops(WORKLOADS["c3"], 4)
    assert vjp == 2 * 512 * 512 * 4096 * 32 and wg == 2 * 512 * (512 + 256) * 4096 * 32
    vjp, _ = bench.algorithmic_flops(WORKLOADS["c4"], 4)
    n, d, s = 16384, 768, 1024
    assert vjp == 24 * (8 * d * d * n + 5 * s * d * n + 16 * d * d * n)
    assert abs(vjp / 7.11e12 - 1) < 2e-3
    # the forward pass of an MLP stack is the same two GEMMs per block
    assert bench.forward_flops(WORKLOADS["c2"]) == 4 * 1024 * 4096 * 8192 * 64


@pytest.mark.parametrize("key,workload", [("gemm_vjp", "c5"), ("gemm_vjp", "c2"), ("scan_lnstat", "c5"),
                                          ("scan_lnstat", "c2"), ("scan_ring", "c3")])
def test_profiled_traffic_belongs_to_the_current_kernels(key, workload):
    """Every entry of the traffic table names the sources it was captured from and their hash; bench.py reports
    `traffic` only while they still match.  A kernel edit without a fresh capture shows up here."""
    t = bench.measured_traffic(key, WORKLOADS[workload])
    assert t is not None, f"{key}: sources changed since the capture in {[e['profile'] for e in bench.TRAFFIC[key]]}"
    assert os.path.exists(os.path.join(ROOT, t["profile"]))


def test_profiled_traffic_is_not_used_for_other_shapes():
    assert bench.measured_traffic("gemm_vjp", WORKLOADS["c4"]) is None
    assert bench.measured_traffic("scan_ring", WORKLOADS["g1"]) is None


def test_config_names_the_workload_and_says_how_l2_is_handled():
    c = bench.config_of(WORKLOADS["c5"], 4, touched_bytes=110e9)
    assert c["workload"].startswith("c5") and c["k"] == 4 and "larger_than_l2" in c["l2"]
    assert bench.config_of(WORKLOADS["c5"], 4) == c          # the reference arm prints the same config
    assert "NOT larger" in bench.config_of(WORKLOADS["c1"], 4, touched_bytes=2e6)["l2"]


def test_reference_arm_prints_the_contract_line():
    """`--impl reference` times the oracle on the host cores and prints one JSON line with the same metric, unit and
    config as the GPU arm, `impl`, a `cpu_baseline` that describes the run and an `e2e` that repeats its value."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["higher_is_better"] is False and line["value"] > 0
    assert line["config"] == bench.config_of(WORKLOADS["c1"], 4)
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["cpu_baseline"]["value"] == line["value"] == line["e2e"]["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
