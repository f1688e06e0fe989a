"""Host-side checks that need no GPU: the library loads, exports every symbol declared in include/hbp.h,
sizes workspaces and rejects bad arguments with status codes."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2501_17086_b200.build import build_library
    build_library()
    from paper_2501_17086_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    header = open(os.path.join(ROOT, "include", "hbp.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(hbp_[a-z0-9_]+)\s*\(", header))
    assert {"hbp_forward", "hbp_backward", "hbp_exact", "hbp_cumsumprod", "hbp_cumsumprod_static"} <= declared
    for name in declared:
        assert hasattr(B.lib, name), name
    assert declared == set(B.EXPORTS)


def test_struct_layout_matches_header(B):
    assert C.sizeof(B.hbp_config) == 64
    assert C.sizeof(B.hbp_params) == 9 * 8 and C.sizeof(B.hbp_grads) == 9 * 8


def test_workspace_sizes_and_config_errors(B):
    c2 = B.make_config("preln_mlp", "bf16", 64, 1024, 8192, hidden=4096)
    c5 = B.make_config("preln_mlp", "bf16", 128, 2048, 16384, hidden=8192)
    n2, n5 = B.workspace_bytes(c2), B.workspace_bytes(c5)
    assert 10 * 2**30 < n2 < 20 * 2**30
    assert n5 < 110 * 2**30          # leaves room for weights, states and gradients on a 180 GB part
    bad = [
        B.make_config("preln_mlp", "bf16", 64, 1020, 8192, hidden=4096),      # d not a multiple of 8
        B.make_config("preln_mlp", "bf16", 0, 1024, 8192, hidden=4096),       # no steps
        B.make_config("rnn_tanh", "f32", 16, 64, 4, in_dim=6, batch=4),        # in_dim not a multiple of 4
        B.make_config("preln_transformer", "bf16", 2, 128, 400, hidden=512, n_heads=3, head_dim=64, seq=200, batch=2),
    ]
    for cfg in bad:
        with pytest.raises(B.HbpError) as e:
            B.workspace_bytes(cfg)
        assert e.value.code == 2
    cfg = B.make_config("preln_mlp", "bf16", 4, 64, 8, hidden=64)
    cfg.dtype = 7
    with pytest.raises(B.HbpError) as e:
        B.workspace_bytes(cfg)
    assert e.value.code == 3
    cfg = B.make_config("preln_transformer", "bf16", 2, 96, 400, hidden=512, n_heads=2, head_dim=48, seq=200, batch=2)
    with pytest.raises(B.HbpError) as e:
        B.workspace_bytes(cfg)
    assert e.value.code == 6


def test_argument_errors_before_any_cuda_call(B):
    lib = B.lib
    n = C.c_size_t()
    assert lib.hbp_workspace_bytes(None, C.byref(n)) == 1
    assert lib.hbp_cumsumprod_scratch_bytes(0, 100, 4, 6, C.byref(n)) == 2     # d % 4
    assert lib.hbp_cumsumprod_scratch_bytes(5, 100, 4, 8, C.byref(n)) == 3
    assert lib.hbp_cumsumprod_scratch_bytes(0, 4096, 32, 512, C.byref(n)) == 0
    assert n.value == 2 * 128 * 32 * 512 * 8                                   # chunk sums and gate products in double
    assert lib.hbp_cumsumprod_scratch_bytes(1, 64, 8192, 1024, C.byref(n)) == 0 and n.value == 0
    assert lib.hbp_cumsumprod(0, 0, 0, 16, 4, 8, None, None, None, None, None, 0, None) == 1   # no delta / g
    assert lib.hbp_forward(None, None, None, None, None, None) == 1
    assert lib.hbp_backward(None, None, 1, None, None, None, None, None, None) == 1
    assert lib.hbp_sync_status(None, None) == 1
    assert B.status_string(8) == "bounded device wait expired"
    assert B.cumsumprod_static_max_bytes() == 32 << 20


def test_relu_residual_kind_is_float_only(B):
    n = C.c_size_t()
    ok = B.make_config("relu_mlp", "f32", 4, 64, 32, hidden=128)
    bad = B.make_config("relu_mlp", "bf16", 4, 64, 32, hidden=128)
    assert B.lib.hbp_workspace_bytes(C.byref(ok), C.byref(n)) == 0 and n.value > 0
    assert B.lib.hbp_workspace_bytes(C.byref(bad), C.byref(n)) == 6


def test_new_entry_points_reject_bad_arguments_without_a_gpu(B):
    lib = B.lib
    assert lib.hbp_iterate(None, None, None, None, None, None, None) == 1
    assert lib.hbp_param_grads(None, None, None, None, None, None, None) == 1
    assert lib.hbp_add_carry(None, None, None, None) == 1
    assert lib.hbp_compare(7, 1, 8, None, None, None, None, 0, None) == 3      # dtype
    assert lib.hbp_compare(0, 0, 8, None, None, None, None, 0, None) == 2      # no segments
    assert lib.hbp_compare(0, 1, 8, None, None, None, None, 0, None) == 1      # null tensors
    assert lib.hbp_compare_scratch_bytes(3) == 3 * 64 * 4 * 8
    n = C.c_size_t()
    for block, kw in (("gru", dict(in_dim=8, batch=4)), ("lstm", dict(hidden=32, in_dim=8, batch=4)),
                      ("postln_mlp", dict(hidden=128))):
        cfg = B.make_config(block, "f32", 6, 64, 4, **kw)
        assert lib.hbp_workspace_bytes(C.byref(cfg), C.byref(n)) == 0 and n.value > 0, block
    bad = B.make_config("lstm", "f32", 6, 64, 4, hidden=20, in_dim=8, batch=4)   # hidden must be d / 2
    assert lib.hbp_workspace_bytes(C.byref(bad), C.byref(n)) == 2
    gated = B.make_config("gru", "f32", 6, 64, 4, in_dim=8, batch=4, gate=B.GATE_CHANNEL_SHARED)
    assert lib.hbp_workspace_bytes(C.byref(gated), C.byref(n)) == 6              # the cell's gate is the only one


def test_diagnostic_entry_points_reject_bad_arguments_without_a_gpu(B):
    lib = B.lib
    assert lib.hbp_context_modes(None) == 0
    assert lib.hbp_selftest_wait_timeout(None, None, 0, 1000000, None) == 1
    # the scan with a status word: same argument checks as the plain one, plus the word's alignment
    assert lib.hbp_cumsumprod_status(0, 0, 0, 16, 4, 8, None, None, None, None, None, 0, None, None) == 1
    assert lib.hbp_cumsumprod_status(0, 0, 0, 16, 4, 8, None, None, None, None, None, 0, C.c_void_p(2), None) == 2
