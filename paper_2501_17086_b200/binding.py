"""ctypes binding over libhbp.so: argument marshalling only.

torch is used for device memory and streams; every step of the path runs in
the library's CUDA kernels.  Importing this module without a built
``libhbp.so`` raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhbp.so")

HBP_F32, HBP_BF16 = 0, 1
BLOCKS = {"mlp": 0, "preln_mlp": 1, "rnn_tanh": 2, "preln_transformer": 3, "gru": 4, "lstm": 5, "relu_mlp": 6, "postln_mlp": 7}
GATE_ONE, GATE_CHANNEL_SHARED, GATE_CHANNEL_PER_STEP = 0, 1, 2
LOSS_FINAL, LOSS_EVERY_STEP = 0, 1

EXPORTS = ["hbp_workspace_bytes", "hbp_create", "hbp_forward", "hbp_backward", "hbp_exact",
           "hbp_cumsumprod_scratch_bytes", "hbp_cumsumprod", "hbp_cumsumprod_status", "hbp_sync_status", "hbp_launch_count",
           "hbp_context_modes", "hbp_selftest_wait_timeout",
           "hbp_profile_enable", "hbp_profile_read", "hbp_cumsumprod_static", "hbp_cumsumprod_static_max_bytes",
           "hbp_compare_scratch_bytes", "hbp_compare", "hbp_iterate", "hbp_add_carry", "hbp_param_grads",
           "hbp_status_string", "hbp_destroy"]


class HbpError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: hbp status {self.code} ({status_string(self.code)})")


class hbp_config(C.Structure):
    _fields_ = [("block", C.c_int32), ("dtype", C.c_int32), ("gate", C.c_int32), ("loss", C.c_int32),
                ("L", C.c_int32), ("d", C.c_int32), ("hidden", C.c_int32), ("in_dim", C.c_int32),
                ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("seq", C.c_int32), ("batch", C.c_int32),
                ("tokens", C.c_int64), ("ln_eps", C.c_float), ("gamma", C.c_float)]


class hbp_params(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("W1", "W2", "W", "U", "Wq", "Wk", "Wv", "Wo", "a")]


class hbp_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("dW1", "dW2", "dW", "dU", "dWq", "dWk", "dWv", "dWo", "da")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2501_17086_b200.build` "
                          "(the library has no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.hbp_workspace_bytes.argtypes = [C.POINTER(hbp_config), C.POINTER(sz)]
    lib.hbp_create.argtypes = [C.POINTER(hbp_config), vp, sz, C.POINTER(vp)]
    lib.hbp_forward.argtypes = [vp, C.POINTER(hbp_params), vp, vp, vp, vp]
    lib.hbp_backward.argtypes = [vp, C.POINTER(hbp_params), i32, vp, vp, vp, vp, C.POINTER(hbp_grads), vp]
    lib.hbp_exact.argtypes = [vp, C.POINTER(hbp_params), vp, vp, vp, vp, C.POINTER(hbp_grads), vp]
    lib.hbp_cumsumprod_scratch_bytes.argtypes = [i32, i32, i64, i32, C.POINTER(sz)]
    lib.hbp_cumsumprod.argtypes = [i32, i32, i32, i32, i64, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.hbp_cumsumprod_status.argtypes = [i32, i32, i32, i32, i64, i32, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.hbp_selftest_wait_timeout.argtypes = [vp, vp, sz, C.c_uint64, vp]
    lib.hbp_context_modes.argtypes = [vp]
    lib.hbp_context_modes.restype = i32
    lib.hbp_cumsumprod_static.argtypes = [i32, i32, i32, i32, i64, i32, vp, vp, vp, vp, vp]
    lib.hbp_cumsumprod_static_max_bytes.argtypes = []
    lib.hbp_iterate.argtypes = [vp, C.POINTER(hbp_params), vp, vp, vp, vp, vp]
    lib.hbp_add_carry.argtypes = [vp, vp, vp, vp]
    lib.hbp_param_grads.argtypes = [vp, C.POINTER(hbp_params), vp, vp, vp, C.POINTER(hbp_grads), vp]
    lib.hbp_compare_scratch_bytes.argtypes = [i32]
    lib.hbp_compare.argtypes = [i32, i32, i64, vp, vp, vp, vp, sz, vp]
    lib.hbp_sync_status.argtypes = [vp, vp]
    lib.hbp_profile_enable.argtypes = [vp, i32]
    lib.hbp_profile_read.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(i64)]
    lib.hbp_launch_count.argtypes = [vp]
    lib.hbp_launch_count.restype = i64
    lib.hbp_status_string.argtypes = [C.c_int]
    lib.hbp_status_string.restype = C.c_char_p
    lib.hbp_destroy.argtypes = [vp]
    lib.hbp_destroy.restype = None
    for name in EXPORTS:
        if name in ("hbp_cumsumprod_static_max_bytes", "hbp_compare_scratch_bytes"):
            getattr(lib, name).restype = sz
        elif name not in ("hbp_launch_count", "hbp_status_string", "hbp_destroy", "hbp_context_modes"):
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


def status_string(code: int) -> str:
    return lib.hbp_status_string(int(code)).decode()


def _check(code, where):
    if code != 0:
        raise HbpError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(dt):
    if dt == torch.float32:
        return HBP_F32
    if dt == torch.bfloat16:
        return HBP_BF16
    raise HbpError(3, "dtype")


def make_config(block, dtype, L, d, tokens, hidden=0, in_dim=0, n_heads=0, head_dim=0, seq=0, batch=0,
                gate=GATE_ONE, loss=LOSS_FINAL, ln_eps=1e-5, gamma=0.0) -> hbp_config:
    return hbp_config(BLOCKS[block], HBP_F32 if dtype in ("f32", torch.float32) else HBP_BF16, gate, loss, L, d,
                      hidden, in_dim, n_heads, head_dim, seq, batch, tokens, ln_eps, gamma)


def config_from_workload(w) -> hbp_config:
    """hbp_config of a ``workloads.Workload``."""
    gate = GATE_CHANNEL_SHARED if w.block == "rnn_tanh" else GATE_ONE
    loss = LOSS_EVERY_STEP if w.loss == "every_mse" else LOSS_FINAL
    return make_config(w.block, w.dtype, w.L, w.d, w.tokens, w.hidden, w.in_dim, w.n_heads, w.head_dim, w.seq,
                       w.batch, gate, loss, w.ln_eps, getattr(w, "gamma", 0.0))


def workspace_bytes(cfg: hbp_config) -> int:
    n = C.c_size_t(0)
    _check(lib.hbp_workspace_bytes(C.byref(cfg), C.byref(n)), "hbp_workspace_bytes")
    return n.value


_GRAD_SHAPES = {
    "mlp": lambda c: {"dW1": (c.L, c.hidden, c.d), "dW2": (c.L, c.d, c.hidden)},
    "rnn_tanh": lambda c: {"dW": (c.d, c.d), "dU": (c.d, c.in_dim)},
    "gru": lambda c: {"dW": (3 * c.d, c.d), "dU": (3 * c.d, c.in_dim)},
    "lstm": lambda c: {"dW": (4 * c.hidden, c.hidden), "dU": (4 * c.hidden, c.in_dim)},
    "preln_transformer": lambda c: {"dW1": (c.L, c.hidden, c.d), "dW2": (c.L, c.d, c.hidden),
                                    **{n: (c.L, c.d, c.d) for n in ("dWq", "dWk", "dWv", "dWo")}},
}
_GRAD_SHAPES["preln_mlp"] = _GRAD_SHAPES["relu_mlp"] = _GRAD_SHAPES["postln_mlp"] = _GRAD_SHAPES["mlp"]
_BLOCK_NAMES = {v: k for k, v in BLOCKS.items()}


class Context:
    """One hbp_ctx over a torch-allocated workspace on the current CUDA device."""

    def __init__(self, cfg: hbp_config, device="cuda"):
        self.cfg = cfg
        self.device = torch.device(device)
        self.dtype = torch.float32 if cfg.dtype == HBP_F32 else torch.bfloat16
        self.block = _BLOCK_NAMES[cfg.block]
        self.steps = 2 * cfg.L if self.block == "preln_transformer" else cfg.L
        nbytes = workspace_bytes(cfg)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        handle = C.c_void_p()
        _check(lib.hbp_create(C.byref(cfg), C.c_void_p(base), nbytes, C.byref(handle)), "hbp_create")
        self._h = handle
        self._keep = None

    def selftest_wait_timeout(self, limit_ns=1_000_000):
        """Enqueues a GEMM tile whose pipeline stalls on purpose with every wait limited to ``limit_ns``; the next
        sync_status() raises HbpError(8)."""
        scratch = torch.empty((128 << 10) + 256, dtype=torch.uint8, device=self.device)
        base = (scratch.data_ptr() + 255) // 256 * 256
        _check(lib.hbp_selftest_wait_timeout(self._h, C.c_void_p(base), 128 << 10, limit_ns, _stream()),
               "hbp_selftest_wait_timeout")
        self._keep = scratch

    @property
    def modes(self) -> int:
        """Bit 0: CUDA-core kernels forced; bit 1: paired-CTA GEMM; bit 2: the scan writes the next VJP's operand
        (float tanh RNN).  Fixed at creation, per context."""
        return int(lib.hbp_context_modes(self._h))

    def close(self):
        if self._h is not None:
            lib.hbp_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- marshalling ----------------------------------------------------
    def _params(self, params):
        p = hbp_params()
        for name, _ in hbp_params._fields_:
            t = params.get(name)
            if t is not None:
                assert t.is_cuda and t.is_contiguous() and t.dtype == self.dtype, name
                setattr(p, name, t.data_ptr())
        return p

    def new_grads(self, with_gate=False):
        c = self.cfg
        out = {n: torch.empty(s, dtype=torch.float32, device=self.device) for n, s in _GRAD_SHAPES[self.block](c).items()}
        if with_gate and c.gate != GATE_ONE:
            out["da"] = torch.empty((c.d,) if c.gate == GATE_CHANNEL_SHARED else (self.steps, c.d),
                                    dtype=torch.float32, device=self.device)
        return out

    def _grads(self, grads):
        if grads is None:
            return None
        g = hbp_grads()
        for name, t in grads.items():
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.float32, name
            setattr(g, name, t.data_ptr())
        return C.byref(g)

    def new_states(self):
        return torch.empty((self.steps + 1, self.cfg.tokens, self.cfg.d), dtype=self.dtype, device=self.device)

    # -- the three calls --------------------------------------------------
    def forward(self, params, x0, inputs=None, x_all=None):
        x_all = self.new_states() if x_all is None else x_all
        p = self._params(params)
        _check(lib.hbp_forward(self._h, C.byref(p), _ptr(x0), _ptr(inputs), _ptr(x_all), _stream()), "hbp_forward")
        return x_all

    def backward(self, params, k, delta, x_all, inputs=None, g_all=None, grads=None):
        g_all = self.new_states() if g_all is None else g_all
        p = self._params(params)
        _check(lib.hbp_backward(self._h, C.byref(p), int(k), _ptr(delta), _ptr(x_all), _ptr(inputs), _ptr(g_all),
                                self._grads(grads), _stream()), "hbp_backward")
        return g_all

    def exact(self, params, delta, x_all, inputs=None, g_all=None, grads=None):
        g_all = self.new_states() if g_all is None else g_all
        p = self._params(params)
        _check(lib.hbp_exact(self._h, C.byref(p), _ptr(delta), _ptr(x_all), _ptr(inputs), _ptr(g_all),
                             self._grads(grads), _stream()), "hbp_exact")
        return g_all

    # -- the pieces of backward, for callers that run the iterations themselves ----------------
    def iterate(self, params, delta, x_all, g_all, inputs=None):
        """One Highway-BP iteration in place on g_all (its last state is read as given, then set to delta_L)."""
        p = self._params(params)
        _check(lib.hbp_iterate(self._h, C.byref(p), _ptr(delta), _ptr(x_all), _ptr(inputs), _ptr(g_all), _stream()),
               "hbp_iterate")
        return g_all

    def add_carry(self, carry, g_all):
        _check(lib.hbp_add_carry(self._h, _ptr(carry), _ptr(g_all), _stream()), "hbp_add_carry")
        return g_all

    def param_grads(self, params, x_all, g_all, grads, inputs=None):
        p = self._params(params)
        _check(lib.hbp_param_grads(self._h, C.byref(p), _ptr(x_all), _ptr(inputs), _ptr(g_all), self._grads(grads),
                                   _stream()), "hbp_param_grads")
        return grads

    def sync_status(self):
        _check(lib.hbp_sync_status(self._h, _stream()), "hbp_sync_status")

    def profile_enable(self, on=True):
        _check(lib.hbp_profile_enable(self._h, 1 if on else 0), "hbp_profile_enable")

    def profile_read(self):
        """{'scan'|'vjp'|'wgrad'|'other': (ms, launches)} since the last read; waits for the recorded events."""
        ms = (C.c_float * 4)()
        n = (C.c_int64 * 4)()
        _check(lib.hbp_profile_read(self._h, ms, n), "hbp_profile_read")
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(("scan", "vjp", "wgrad", "other"))}

    @property
    def launches(self) -> int:
        return int(lib.hbp_launch_count(self._h))


def cumsumprod_scratch_bytes(dtype, L, rows, d) -> int:
    n = C.c_size_t(0)
    _check(lib.hbp_cumsumprod_scratch_bytes(_dtype_code(dtype), L, rows, d, C.byref(n)), "hbp_cumsumprod_scratch_bytes")
    return n.value


def cumsumprod(u, delta, a=None, gate=None, loss=LOSS_FINAL, g=None, scratch=None, status=None):
    """g[L] = delta_L, g[l] = delta_l + a_l * g[l+1] + u[l]; u is [L, rows, d] (or None with ``g`` given).
    ``status``: an int32 device tensor (zeroed by the caller) that receives a kernel's error code, if any."""
    ref = u if u is not None else g
    L = ref.shape[0] - (0 if u is not None else 1)
    rows, d = ref.shape[1], ref.shape[2]
    if gate is None:
        gate = GATE_ONE if a is None else (GATE_CHANNEL_SHARED if a.dim() == 1 else GATE_CHANNEL_PER_STEP)
    if g is None:
        g = torch.empty((L + 1, rows, d), dtype=ref.dtype, device=ref.device)
    need = cumsumprod_scratch_bytes(ref.dtype, L, rows, d)
    if scratch is None and need:
        scratch = torch.empty(need, dtype=torch.uint8, device=ref.device)
    nbytes = 0 if scratch is None else scratch.numel()
    if status is not None:
        _check(lib.hbp_cumsumprod_status(_dtype_code(ref.dtype), gate, loss, L, rows, d, _ptr(u), _ptr(delta), _ptr(a),
                                         _ptr(g), _ptr(scratch), nbytes, _ptr(status), _stream()), "hbp_cumsumprod_status")
        return g
    _check(lib.hbp_cumsumprod(_dtype_code(ref.dtype), gate, loss, L, rows, d, _ptr(u), _ptr(delta), _ptr(a), _ptr(g),
                              _ptr(scratch), nbytes, _stream()), "hbp_cumsumprod")
    return g


def cumsumprod_static_max_bytes() -> int:
    return int(lib.hbp_cumsumprod_static_max_bytes())


def cumsumprod_static(u, delta, a=None, gate=None, loss=LOSS_FINAL, g=None):
    """hbp_cumsumprod for callers that cannot allocate: the scratch of the time-chunked scan lives in a
    fixed 32 MiB array inside the library, so only inputs and the output are passed.  ``g`` must be given
    by such callers (this wrapper makes one with torch only when it is omitted).  Raises HbpError with
    status 5 when the problem needs more scratch than the fixed array holds."""
    L, rows, d = u.shape
    if gate is None:
        gate = GATE_ONE if a is None else (GATE_CHANNEL_SHARED if a.dim() == 1 else GATE_CHANNEL_PER_STEP)
    if g is None:
        g = torch.empty((L + 1, rows, d), dtype=u.dtype, device=u.device)
    _check(lib.hbp_cumsumprod_static(_dtype_code(u.dtype), gate, loss, L, rows, d, _ptr(u), _ptr(delta), _ptr(a),
                                     _ptr(g), _stream()), "hbp_cumsumprod_static")
    return g


def compare(a, b, segments=1):
    """<a,b>, |a|^2, |b|^2, |a-b|^2 per segment of two equally shaped tensors split into ``segments`` consecutive
    blocks (e.g. the states g_l of two estimates): a float64 tensor [segments, 4] on the device.  The cosine
    similarity of Figure 5 is out[:, 0] / sqrt(out[:, 1] * out[:, 2])."""
    assert a.shape == b.shape and a.dtype == b.dtype and a.is_contiguous() and b.is_contiguous()
    assert a.numel() % segments == 0
    out = torch.empty((segments, 4), dtype=torch.float64, device=a.device)
    need = int(lib.hbp_compare_scratch_bytes(segments))
    scratch = torch.empty(need, dtype=torch.uint8, device=a.device)
    _check(lib.hbp_compare(_dtype_code(a.dtype), segments, a.numel() // segments, _ptr(a), _ptr(b), _ptr(out),
                           _ptr(scratch), need, _stream()), "hbp_compare")
    return out
