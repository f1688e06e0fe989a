"""fp64 CPU oracle for Highway backpropagation (arXiv 2501.17086).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the
CUDA library is checked against.  It shares no code with the CUDA path and is
imported only by the tests, by the smoke check and by the CPU-baseline leg of
the benchmark.  The product never routes through it.

Notation.  The paper numbers layers i = 1..L with h_i = f_i(h_{i-1}), h_0 = x
(Section 3) and treats gradients as row vectors multiplied on the left.  Here a
"step" l = 0..L-1 maps state x_l to x_{l+1} = a_l * x_l + f_l(x_l); paper layer
i is step l = i-1, h_i = x_i, K_{l+1} = diag(a_l) and J_{l+1} is the Jacobian of
the block f_l at x_l (Section 3, Eq. 1-2 with r(x, z) = a * x + z).  The local
loss gradient at state l is delta_l (Section 3, the general loss form).

Everything is float64 numpy.  Weight containers may be any object indexable by
the step number whose items convert with ``np.asarray(..., float64)``; they are
converted one step at a time so that very large stacks never need a full
float64 copy.

Pinned by tests/test_oracle_*.py (brute-force path sums of Theorem 1/2, finite
differences, closed forms, special cases).  Numeric values on the synthetic
workloads themselves are "parity unpinned" beyond those pins: the paper prints
no worked example.
"""
from __future__ import annotations

import itertools
import math

import numpy as np
from scipy.special import erf as _erf

_SQRT2 = math.sqrt(2.0)
_INV_SQRT_2PI = 1.0 / math.sqrt(2.0 * math.pi)


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# Elementwise pieces
# --------------------------------------------------------------------------
def gelu(z):
    """Exact (erf) GELU: 0.5 z (1 + erf(z / sqrt 2))."""
    return 0.5 * z * (1.0 + _erf(z / _SQRT2))


def gelu_prime(z):
    """d/dz of the exact GELU: Phi(z) + z * pdf(z)."""
    return 0.5 * (1.0 + _erf(z / _SQRT2)) + z * np.exp(-0.5 * z * z) * _INV_SQRT_2PI


def layernorm(x, eps):
    """LayerNorm without affine over the last axis, biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    return (x - mu) * rstd, rstd


def layernorm_vjp(xhat, rstd, dy):
    """Row-vector VJP of layernorm: rstd (dy - mean dy - xhat mean(dy xhat))."""
    m1 = dy.mean(axis=-1, keepdims=True)
    m2 = (dy * xhat).mean(axis=-1, keepdims=True)
    return rstd * (dy - m1 - xhat * m2)


# --------------------------------------------------------------------------
# Blocks f_l.  Each has forward(x) -> (f, cache), vjp(cache, g) -> J^T g,
# param_vjp(cache, g) -> dict of parameter gradients, all hand-written.
# --------------------------------------------------------------------------
class MLPStep:
    """f(x) = phi(y W1^T) W2^T with y = x, or y = LN(x) for the pre-LN form
    (Table 1, rows "Pre-activation ResNet" / "Transformer (Pre-LN)")."""

    def __init__(self, W1, W2, pre_ln, eps=1e-5):
        self.W1, self.W2, self.pre_ln, self.eps = W1, W2, bool(pre_ln), eps

    def forward(self, x):
        W1, W2 = _f64(self.W1), _f64(self.W2)
        if self.pre_ln:
            y, rstd = layernorm(x, self.eps)
        else:
            y, rstd = x, None
        z = y @ W1.T
        f = gelu(z) @ W2.T
        return f, dict(y=y, rstd=rstd, z=z)

    def _dz(self, cache, g):
        return (g @ _f64(self.W2)) * gelu_prime(cache["z"])

    def vjp(self, cache, g):
        dy = self._dz(cache, g) @ _f64(self.W1)
        if self.pre_ln:
            return layernorm_vjp(cache["y"], cache["rstd"], dy)
        return dy

    def param_vjp(self, cache, g):
        dz = self._dz(cache, g)
        g2 = g.reshape(-1, g.shape[-1])
        a2 = gelu(cache["z"]).reshape(g2.shape[0], -1)
        dz2 = dz.reshape(g2.shape[0], -1)
        y2 = cache["y"].reshape(g2.shape[0], -1)
        return {"W2": g2.T @ a2, "W1": dz2.T @ y2}


class AttnStep:
    """f(x) = MHA(LN(x)) Wo^T, causal softmax attention, x of shape [B, S, d]
    (Table 1, row "Transformer (Pre-LN)"; attention sub-layer of Section 5.1.1)."""

    def __init__(self, Wq, Wk, Wv, Wo, n_heads, eps=1e-5):
        self.Wq, self.Wk, self.Wv, self.Wo = Wq, Wk, Wv, Wo
        self.H, self.eps = int(n_heads), eps

    def _split(self, t):
        B, S, d = t.shape
        return t.reshape(B, S, self.H, d // self.H).transpose(0, 2, 1, 3)

    @staticmethod
    def _merge(t):
        B, H, S, dh = t.shape
        return t.transpose(0, 2, 1, 3).reshape(B, S, H * dh)

    def forward(self, x):
        y, rstd = layernorm(x, self.eps)
        q = self._split(y @ _f64(self.Wq).T)
        k = self._split(y @ _f64(self.Wk).T)
        v = self._split(y @ _f64(self.Wv).T)
        S = x.shape[1]
        scale = 1.0 / math.sqrt(q.shape[-1])
        s = (q @ k.transpose(0, 1, 3, 2)) * scale
        future = np.triu(np.ones((S, S), dtype=bool), 1)
        s = np.where(future, -np.inf, s)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=-1, keepdims=True)
        o = self._merge(p @ v)
        f = o @ _f64(self.Wo).T
        return f, dict(y=y, rstd=rstd, q=q, k=k, v=v, p=p, o=o, scale=scale)

    def _core_vjp(self, c, g):
        do = self._split(g @ _f64(self.Wo))
        p, q, k, v = c["p"], c["q"], c["k"], c["v"]
        dv = p.transpose(0, 1, 3, 2) @ do
        dp = do @ v.transpose(0, 1, 3, 2)
        ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
        dq = (ds @ k) * c["scale"]
        dk = (ds.transpose(0, 1, 3, 2) @ q) * c["scale"]
        return self._merge(dq), self._merge(dk), self._merge(dv)

    def vjp(self, c, g):
        dq, dk, dv = self._core_vjp(c, g)
        dy = dq @ _f64(self.Wq) + dk @ _f64(self.Wk) + dv @ _f64(self.Wv)
        return layernorm_vjp(c["y"], c["rstd"], dy)

    def param_vjp(self, c, g):
        dq, dk, dv = self._core_vjp(c, g)
        d = g.shape[-1]
        y2 = c["y"].reshape(-1, d)
        return {
            "Wo": g.reshape(-1, d).T @ c["o"].reshape(-1, d),
            "Wq": dq.reshape(-1, d).T @ y2,
            "Wk": dk.reshape(-1, d).T @ y2,
            "Wv": dv.reshape(-1, d).T @ y2,
        }


class RNNStep:
    """f_t(h) = tanh(h W^T + x_t U^T): one cell of a recurrent network seen as
    a layer whose parameters are [theta, x_t] (Section 5.2)."""

    def __init__(self, W, U, x_t):
        self.W, self.U, self.x_t = W, U, x_t

    def forward(self, h):
        c = np.tanh(h @ _f64(self.W).T + _f64(self.x_t) @ _f64(self.U).T)
        return c, dict(c=c, h=h)

    def vjp(self, cache, g):
        return (g * (1.0 - cache["c"] ** 2)) @ _f64(self.W)

    def param_vjp(self, cache, g):
        dz = g * (1.0 - cache["c"] ** 2)
        return {"W": dz.T @ cache["h"], "U": dz.T @ _f64(self.x_t)}


def _sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


class GRUStep:
    """One GRU cell as a layer with a data-dependent gate (Table 1, row "GRU": f(x) = a(x) * x + b(x),
    g = [a, b], r(x, z) = z1 * x + z2).  With r = sigmoid(U_r x_t + W_r h), z = sigmoid(U_z x_t + W_z h),
    n = tanh(U_n x_t + r * (W_n h)):  h' = z * h + (1 - z) * n, so a(h) = z, b(h) = (1 - z) * n,
    K = diag(z) and J = diag(h) da/dh + db/dh.  W [3d, d] and U [3d, in] stack the r, z, n rows."""

    def __init__(self, W, U, x_t):
        self.W, self.U, self.x_t = W, U, x_t

    def forward(self, h):
        W, U = _f64(self.W), _f64(self.U)
        d = h.shape[-1]
        pre = _f64(self.x_t) @ U.T
        rec = h @ W.T
        r = _sigmoid(pre[..., :d] + rec[..., :d])
        z = _sigmoid(pre[..., d:2 * d] + rec[..., d:2 * d])
        rec_n = rec[..., 2 * d:]
        n = np.tanh(pre[..., 2 * d:] + r * rec_n)
        return (1.0 - z) * n, dict(h=h, r=r, z=z, n=n, rec_n=rec_n)

    def gate(self, cache):
        return cache["z"]

    def _pre_grads(self, c, g):
        dn_pre = g * (1.0 - c["z"]) * (1.0 - c["n"] ** 2)
        dz_pre = g * (c["h"] - c["n"]) * c["z"] * (1.0 - c["z"])      # through a = z (times h) and through b
        dr_pre = dn_pre * c["rec_n"] * c["r"] * (1.0 - c["r"])
        return dr_pre, dz_pre, dn_pre

    def vjp(self, c, g):
        dr_pre, dz_pre, dn_pre = self._pre_grads(c, g)
        return np.concatenate([dr_pre, dz_pre, dn_pre * c["r"]], axis=-1) @ _f64(self.W)

    def param_vjp(self, c, g):
        dr_pre, dz_pre, dn_pre = self._pre_grads(c, g)
        rec = np.concatenate([dr_pre, dz_pre, dn_pre * c["r"]], axis=-1)
        pre = np.concatenate([dr_pre, dz_pre, dn_pre], axis=-1)
        return {"W": rec.T @ c["h"], "U": pre.T @ _f64(self.x_t)}


class LSTMStep:
    """One LSTM cell as a layer on the state x = [c, h] (Table 1, row "LSTM": f(x) = [a(x) * x_c + b(x), c(x)],
    r(x, z) = [z1 * x_c + z2, z3]).  With [i, f, g, o] = [sigmoid, sigmoid, tanh, sigmoid](U x_t + W h):
    c' = f * c + i * g,  h' = o * tanh(c').  The residual Jacobian is K = diag([f, 0]): only the cell state has a
    linear path; everything else, including the path from c to h' through tanh(c'), belongs to J.
    W [4u, u] and U [4u, in] stack the i, f, g, o rows (u = units; the state is 2u wide)."""

    def __init__(self, W, U, x_t):
        self.W, self.U, self.x_t = W, U, x_t

    def forward(self, x):
        W, U = _f64(self.W), _f64(self.U)
        u = x.shape[-1] // 2
        c, h = x[..., :u], x[..., u:]
        pre = _f64(self.x_t) @ U.T + h @ W.T
        i, f, o = _sigmoid(pre[..., :u]), _sigmoid(pre[..., u:2 * u]), _sigmoid(pre[..., 3 * u:])
        g = np.tanh(pre[..., 2 * u:3 * u])
        c_new = f * c + i * g
        tc = np.tanh(c_new)
        h_new = o * tc
        block = np.concatenate([i * g, h_new], axis=-1)          # what r adds to the gated state
        return block, dict(c=c, h=h, i=i, f=f, g=g, o=o, tc=tc)

    def gate(self, cache):
        return np.concatenate([cache["f"], np.zeros_like(cache["f"])], axis=-1)

    def _pre_grads(self, k, g):
        u = k["f"].shape[-1]
        gc, gh = g[..., :u], g[..., u:]
        through_h = gh * k["o"] * (1.0 - k["tc"] ** 2)           # dLoss/dc' that arrives through h' = o tanh(c')
        dct = gc + through_h
        pre = np.concatenate([dct * k["g"] * k["i"] * (1.0 - k["i"]), dct * k["c"] * k["f"] * (1.0 - k["f"]),
                              dct * k["i"] * (1.0 - k["g"] ** 2), gh * k["tc"] * k["o"] * (1.0 - k["o"])], axis=-1)
        return pre, through_h

    def vjp(self, k, g):
        pre, through_h = self._pre_grads(k, g)
        # the cell state's share of J: f * (what came through h'); f * g_c itself is K's
        return np.concatenate([k["f"] * through_h, pre @ _f64(self.W)], axis=-1)

    def param_vjp(self, k, g):
        pre, _ = self._pre_grads(k, g)
        return {"W": pre.T @ k["h"], "U": pre.T @ _f64(self.x_t)}


class ReluResStep:
    """ResNet-style layer f(x) = ReLU(x + Block(x)) (Table 1, row "ResNet": g = Block, r(x, z) = ReLU(x + z)).
    dr/dx = dr/dz = diag(mask) with mask = [x + Block(x) > 0], so K = diag(mask) depends on the state and
    J = diag(mask) J_Block.  `inner` is the block (an MLPStep)."""

    def __init__(self, inner):
        self.inner = inner

    def forward(self, x):
        z, cache = self.inner.forward(x)
        mask = (x + z > 0.0).astype(np.float64)
        cache = dict(cache)
        cache["mask"] = mask
        return mask * z, cache            # r(x, z) = mask * x + mask * z: the gate carries the first term

    def gate(self, cache):
        return cache["mask"]

    def vjp(self, cache, g):
        return self.inner.vjp(cache, cache["mask"] * g)

    def param_vjp(self, cache, g):
        return self.inner.param_vjp(cache, cache["mask"] * g)


class PostLNStep:
    """Post-LayerNorm layer f(x) = LN(x + Block(x)) (Table 1, row "Transformer (Post-LN)": g = [a(x), b(x)],
    r(x, z) = z1 * x + z2; Appendix C.3's derivation with alpha = 1, beta = 0): with y = x + Block(x),
    a(x) = 1 / sigma(y) per row and b(x) = (Block(x) - mu(y)) / sigma(y).  K = diag(a) is a row-wise scalar gate that
    depends on the state; J is the rest of the layer's Jacobian.  `inner` is the block (an MLPStep).
    With the shift gamma of Appendix C.3 the split is g = [(1 - gamma) a, b + gamma x a]: K = (1 - gamma) diag(a), the
    layer itself (and exact backpropagation) unchanged."""

    def __init__(self, inner, eps, gamma=0.0):
        self.inner, self.eps, self.gamma = inner, eps, float(gamma)

    def forward(self, x):
        z, cache = self.inner.forward(x)
        out, rstd = layernorm(x + z, self.eps)
        cache = dict(cache)
        cache["out"], cache["rstd"] = out, rstd
        return out - (1.0 - self.gamma) * rstd * x, cache      # what r adds to the gated state

    def gate(self, cache):
        return (1.0 - self.gamma) * cache["rstd"]              # [..., 1]: the same gate for every channel of a row

    def _through_ln(self, cache, g):
        return layernorm_vjp(cache["out"], cache["rstd"], g)

    def vjp(self, cache, g):
        t = self._through_ln(cache, g)    # dLoss/dy; the layer's full VJP is t + J_Block^T t
        return t - (1.0 - self.gamma) * cache["rstd"] * g + self.inner.vjp(cache, t)

    def param_vjp(self, cache, g):
        return self.inner.param_vjp(cache, self._through_ln(cache, g))


class ShiftedStep:
    """The gamma-shifted split of a residual layer x + Block(x) (Appendix C.3, Eq. 17): the block becomes
    g(x) = Block(x) + gamma x and the residual function r(x, z) = (1 - gamma) x + z, so the layer itself is
    unchanged while J gains gamma I and K becomes (1 - gamma) I."""

    def __init__(self, step, gamma):
        self.step, self.gamma = step, float(gamma)

    def forward(self, x):
        f, cache = self.step.forward(x)
        return f + self.gamma * x, cache

    def vjp(self, cache, g):
        return self.step.vjp(cache, g) + self.gamma * g

    def param_vjp(self, cache, g):
        return self.step.param_vjp(cache, g)


def shifted_stack(stack, gamma):
    """Same network as ``stack`` (all gates 1), split with the shift gamma."""
    if any(a is not None for a in stack.gates):
        raise ValueError("the shift is defined for plain residual connections")
    return Stack([ShiftedStep(st, gamma) for st in stack.steps], [1.0 - float(gamma)] * stack.L)


class Stack:
    """L residual steps x_{l+1} = a_l * x_l + f_l(x_l).

    ``gates[l]`` is None (a_l = 1), a scalar, or a per-channel vector [d]: the
    diagonal of K_{l+1} (Eq. 2).  ``names[l]`` tells which parameter group the
    step's gradients accumulate into: (group, index) with index None for
    weights shared by all steps."""

    def __init__(self, steps, gates=None, names=None, gate_shared=False):
        self.steps = list(steps)
        self.L = len(self.steps)
        self.gates = list(gates) if gates is not None else [None] * self.L
        self.names = names
        self.gate_shared = gate_shared

    def gate(self, l, caches=None):
        """Diagonal of K_{l+1}: a constant, or - for blocks with a data-dependent gate (GRU) - the value the
        forward pass produced at x_l, taken from its cache."""
        step = self.steps[l]
        if hasattr(step, "gate"):
            if caches is None:
                raise ValueError("this stack's gates depend on the states: pass the forward caches")
            return step.gate(caches[l])
        a = self.gates[l]
        return 1.0 if a is None else _f64(a)


def mlp_stack(W1, W2, pre_ln, eps=1e-5, gate=None):
    L = len(W1)
    steps = [MLPStep(_Lazy(W1, l), _Lazy(W2, l), pre_ln, eps) for l in range(L)]
    return Stack(steps, [gate] * L)


def gru_stack(W, U, X):
    """GRU over time; X is [T, B, in]."""
    T = len(X)
    return Stack([GRUStep(W, U, _Lazy(X, t)) for t in range(T)])


def lstm_stack(W, U, X):
    """LSTM over time on the state [c, h]; X is [T, B, in]."""
    return Stack([LSTMStep(W, U, _Lazy(X, t)) for t in range(len(X))])


def relu_mlp_stack(W1, W2):
    """L layers x <- ReLU(x + W2 gelu(W1 x))."""
    return Stack([ReluResStep(s) for s in mlp_stack(W1, W2, False, 0.0).steps])


def postln_mlp_stack(W1, W2, eps=1e-5, gamma=0.0):
    """L layers x <- LN(x + W2 gelu(W1 x)), LayerNorm without affine; gamma = the shift of the split."""
    return Stack([PostLNStep(s, eps, gamma) for s in mlp_stack(W1, W2, False, 0.0).steps])


def rnn_stack(W, U, a, X):
    """Gated tanh RNN: h_{t+1} = a * h_t + tanh(W h_t + U x_t); X is [T, B, in]."""
    T = len(X)
    steps = [RNNStep(W, U, _Lazy(X, t)) for t in range(T)]
    return Stack(steps, [a] * T, gate_shared=True)


def transformer_stack(Wq, Wk, Wv, Wo, W1, W2, n_heads, eps=1e-5):
    """Each decoder block is two residual steps, attention then MLP
    (Section 5.1.1: layers split into two sub-layers)."""
    steps = []
    for b in range(len(Wq)):
        steps.append(AttnStep(_Lazy(Wq, b), _Lazy(Wk, b), _Lazy(Wv, b), _Lazy(Wo, b), n_heads, eps))
        steps.append(MLPStep(_Lazy(W1, b), _Lazy(W2, b), True, eps))
    return Stack(steps)


class _Lazy:
    """Defers ``container[index]`` (and its float64 conversion) until used."""

    def __init__(self, container, index):
        self.container, self.index = container, index

    def __array__(self, dtype=None, copy=None):
        a = np.asarray(self.container[self.index], dtype=np.float64)
        return a if dtype is None else a.astype(dtype, copy=False)


# --------------------------------------------------------------------------
# The method
# --------------------------------------------------------------------------
def forward(stack, x0):
    """Section 3: h_i = f_i(h_{i-1}).  Returns states x_0..x_L and the caches."""
    xs, caches = [_f64(x0)], []
    for l, step in enumerate(stack.steps):
        f, cache = step.forward(xs[l])
        caches.append(cache)
        xs.append(stack.gate(l, caches) * xs[l] + f)
    return xs, caches


def exact_bp(stack, caches, deltas):
    """Plain chain rule (Section 2.2; first line of the proof of Theorem 1):
    g_L = delta_L, g_l = delta_l + (J_{l+1} + K_{l+1})^T g_{l+1}."""
    L = stack.L
    g = [None] * (L + 1)
    g[L] = _f64(deltas[L])
    for l in range(L - 1, -1, -1):
        g[l] = _f64(deltas[l]) + stack.gate(l, caches) * g[l + 1] + stack.steps[l].vjp(caches[l], g[l + 1])
    return g


def cumsumprod_sequential(v, gates):
    """The recurrence of Eq. 9, u_i = v_i + u_{i+1} K_{i+1}, solved in order.

    ``v`` holds v_0..v_{n-1}; ``gates[i]`` is the diagonal of K_{i+1} (a scalar
    or vector); the term beyond the last index is zero."""
    n = len(v)
    u = [None] * n
    u[n - 1] = _f64(v[n - 1])
    for i in range(n - 2, -1, -1):
        u[i] = _f64(v[i]) + _f64(gates[i]) * u[i + 1]
    return u


def cumsumprod_definition(v, gates):
    """Eq. 12 written out: CumSumProd(a, M)_i = sum_{j>=i} a_j M_j ... M_{i+1}."""
    n = len(v)
    out = []
    for i in range(n):
        acc = np.zeros_like(_f64(v[i]))
        for j in range(i, n):
            term = _f64(v[j])
            for m in range(j - 1, i - 1, -1):  # apply K_j, then K_{j-1}, ... K_{i+1}
                term = term * _f64(gates[m])
            acc = acc + term
        out.append(acc)
    return out


def cumsumprod_parallel(v, K):
    """Algorithm 1 (reversed Hillis-Steele scan), ceil(log2 n) rounds.

    ``v`` holds v_1..v_n (index 0 is v_1).  ``K[i]`` is the matrix that carries
    a row vector at position i+1 back to position i, i.e. the paper's K_{i+1}
    as seen from position i; it may be a scalar / vector (diagonal K) or a
    dense matrix with v_{i+1} @ K[i] defined.  The printed initialisation
    P <- K does not type-check against the algorithm's own post-condition; the
    reading taken is P_i^{(0)} = K_{i+1}, which does, and the slot for the last
    position is never read for a result."""
    n = len(v)
    u = [_f64(x) for x in v]
    P = [(_f64(K[i]) if i < n - 1 else None) for i in range(n)]

    def apply(vec, mat):
        return vec @ mat if (np.ndim(mat) == 2) else vec * mat

    def compose(far, near):
        # (K_{..far block..})(K_{..near block..}): far applied first to a row vector
        if far is None or near is None:
            return None
        if np.ndim(far) == 2 and np.ndim(near) == 2:
            return far @ near
        return far * near  # both diagonal (scalars or vectors)

    M = max(0, math.ceil(math.log2(n))) if n > 1 else 0
    for m in range(M):
        s = 1 << m
        nu, nP = list(u), list(P)
        for i in range(n):
            if i + s <= n - 1:
                nu[i] = u[i] + apply(u[i + s], P[i])
                nP[i] = compose(P[i + s], P[i])
        u, P = nu, nP
    return u


def initial_estimate(stack, deltas, caches=None):
    """Eq. 5 / Eq. 10: w^0 = CumSumProd(delta, K), the pure residual-path term."""
    L = stack.L
    w0 = [None] * (L + 1)
    w0[L] = _f64(deltas[L])
    for l in range(L - 1, -1, -1):
        w0[l] = _f64(deltas[l]) + stack.gate(l, caches) * w0[l + 1]
    return w0


def highway_bp(stack, caches, deltas, k, return_all=False):
    """Theorem 2 in the two-step form of Section 4.3, taken literally:
    keep w^0; each iteration computes v_l = J_{l+1}^T w^j_{l+1} for every l from
    the OLD iterate (Eq. 8), solves u_l = v_l + a_l u_{l+1} (Eq. 9) and sets
    w^{j+1}_l = w^0_l + u_l (Eq. 11).  Returns w^k_0..w^k_L."""
    if k < 0:
        raise ValueError("k must be >= 0")
    L = stack.L
    w0 = initial_estimate(stack, deltas, caches)
    w = list(w0)
    history = [list(w)]
    for _ in range(k):
        v = [stack.steps[l].vjp(caches[l], w[l + 1]) for l in range(L)]
        u = cumsumprod_sequential(v, [stack.gate(l, caches) for l in range(L)])
        w = [w0[l] + u[l] for l in range(L)] + [w0[L]]
        history.append(list(w))
    return history if return_all else w


def highway_bp_folded(stack, caches, deltas, k):
    """Same result with delta folded into one scan per iteration,
    g_l = delta_l + a_l g_{l+1} + u_l; equal to the literal form by linearity
    of the recurrence."""
    L = stack.L
    g = initial_estimate(stack, deltas, caches)
    for _ in range(k):
        v = [stack.steps[l].vjp(caches[l], g[l + 1]) for l in range(L)]
        new = [None] * (L + 1)
        new[L] = _f64(deltas[L])
        for l in range(L - 1, -1, -1):
            new[l] = _f64(deltas[l]) + stack.gate(l, caches) * new[l + 1] + v[l]
        g = new
    return g


def param_grads(stack, caches, xs, g, groups):
    """Section 4.2, last sentence: dL/dtheta_i = (dL/dh_i)(df_i/dtheta_i), with
    whatever estimate ``g`` is given in place of the exact gradient.

    ``groups[l]`` = (prefix, index): gradients of step l go to key
    ``prefix + name`` at position ``index`` (a list), or are summed into a
    single array when index is None (weights shared by all steps).  A gate
    that is a trainable per-channel vector gets da = sum g_{l+1} * x_l."""
    out = {}
    for l, step in enumerate(stack.steps):
        prefix, index = groups[l]
        for name, val in step.param_vjp(caches[l], g[l + 1]).items():
            key = prefix + name
            if index is None:
                out[key] = out.get(key, 0.0) + val
            else:
                out.setdefault(key, {})[index] = val
    if stack.gate_shared:
        da = 0.0
        for l in range(stack.L):
            da = da + (g[l + 1] * xs[l]).reshape(-1, xs[l].shape[-1]).sum(axis=0)
        out["a"] = da
    for key, val in list(out.items()):
        if isinstance(val, dict):
            out[key] = np.stack([val[i] for i in sorted(val)])
    return out


# --------------------------------------------------------------------------
# Brute force of the definitions (tiny sizes only)
# --------------------------------------------------------------------------
def finite_difference_jacobian(fn, x, h=1e-6):
    """Central differences of a vector function at a single point x [d]."""
    x = _f64(x)
    cols = []
    for j in range(x.size):
        e = np.zeros_like(x)
        e[j] = h
        cols.append((fn(x + e) - fn(x - e)) / (2.0 * h))
    return np.stack(cols, axis=1)  # [out, in]


def path_sum(deltas, J, K, i, k):
    """Theorem 2's definition of w^k_i: the sum over end points j >= i and over
    subsets of [i+1, j] with at most k elements of G_ij (Eq. 3), each G being
    delta_j times J_m or K_m for m = j down to i+1.  ``J[m]`` and ``K[m]`` are
    dense matrices of the paper's layer m (1-based; index 0 unused)."""
    L = len(J) - 1
    total = np.zeros_like(_f64(deltas[i]))
    for j in range(i, L + 1):
        idx = list(range(i + 1, j + 1))
        for r in range(0, min(k, len(idx)) + 1):
            for subset in itertools.combinations(idx, r):
                chosen = set(subset)
                vec = _f64(deltas[j])
                for m in range(j, i, -1):
                    vec = vec @ (J[m] if m in chosen else K[m])
                total = total + vec
    return total


def agreement(a, b):
    """The four sums behind Figure 5 for two gradient estimates: <a,b>, |a|^2, |b|^2, |a-b|^2 (cosine similarity =
    first / sqrt(second * third); relative size of a step = sqrt(fourth / third))."""
    a, b = _f64(a).reshape(-1), _f64(b).reshape(-1)
    d = a - b
    return np.array([a @ b, a @ a, b @ b, d @ d])
