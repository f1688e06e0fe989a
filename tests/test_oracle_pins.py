"""Pins for the fp64 oracle: what the paper and the mathematics fix.

None of these tests compares the oracle with itself through the same code
path: the references are brute-force path sums over dense Jacobians obtained
by finite differences of the forward function, finite differences of the
scalar loss, closed forms, and library routines.
"""
import math
import os

import numpy as np
import pytest

from oracle import hbp_oracle as O

RNG = np.random.default_rng(7)


# ---------------------------------------------------------------- helpers
class LinearStep:
    """f(x) = x C^T: a block with a constant Jacobian (test-local)."""

    def __init__(self, C):
        self.C = np.atleast_2d(np.asarray(C, dtype=np.float64))

    def forward(self, x):
        return x @ self.C.T, dict(x=x)

    def vjp(self, cache, g):
        return g @ self.C

    def param_vjp(self, cache, g):
        return {"C": g.T @ cache["x"]}


def tiny_stack(kind, L=4, d=3, h=5, gate="vector", rng=RNG):
    if gate == "vector":
        gates = [rng.uniform(0.5, 1.1, size=d) for _ in range(L)]
    elif gate == "one":
        gates = [None] * L
    else:
        gates = [np.zeros(d)] * L
    if kind in ("mlp", "preln_mlp"):
        steps = [O.MLPStep(rng.normal(size=(h, d)) / math.sqrt(d), rng.normal(size=(d, h)) / math.sqrt(h),
                           kind == "preln_mlp") for _ in range(L)]
    elif kind == "rnn":
        W = rng.normal(size=(d, d)) * 0.6
        U = rng.normal(size=(d, 2))
        steps = [O.RNNStep(W, U, rng.normal(size=(1, 2))) for _ in range(L)]
    else:
        raise ValueError(kind)
    return O.Stack(steps, gates)


def dense_jacobians(stack, xs):
    """J_m, K_m (1-based paper layers) by central differences of the forward
    function of each block at the stored state: independent of every VJP."""
    L = stack.L
    J, K = [None], [None]
    for l in range(L):
        shape = xs[l].shape

        def block(xflat, l=l, shape=shape):
            return stack.steps[l].forward(xflat.reshape(shape))[0].reshape(-1)

        J.append(O.finite_difference_jacobian(block, xs[l].reshape(-1), h=1e-5))
        a = np.broadcast_to(stack.gate(l), shape).reshape(-1)
        K.append(np.diag(a))
    return J, K


def random_deltas(xs, every=True, rng=RNG):
    L = len(xs) - 1
    out = [np.zeros_like(xs[0]) for _ in range(L + 1)]
    for l in range(L + 1):
        if every or l == L:
            out[l] = rng.normal(size=xs[l].shape)
    return out


# ------------------------------------------------- 1. brute force of Thm 1/2
@pytest.mark.parametrize("kind", ["mlp", "preln_mlp", "rnn"])
@pytest.mark.parametrize("gate", ["vector", "one"])
def test_truncated_path_sum_equals_iteration(kind, gate):
    L = 5
    stack = tiny_stack(kind, L=L, gate=gate)
    xs, caches = O.forward(stack, RNG.normal(size=(1, 3)))
    deltas = random_deltas(xs, every=True)
    J, K = dense_jacobians(stack, xs)
    flat = [d.reshape(-1) for d in deltas]
    hist = O.highway_bp(stack, caches, deltas, L, return_all=True)
    for k in range(L + 1):
        for i in range(L + 1):
            ref = O.path_sum(flat, J, K, i, k)
            np.testing.assert_allclose(hist[k][i].reshape(-1), ref, rtol=1e-6, atol=1e-8)
    # all 2^L paths = the exact gradient (Theorem 1)
    g = O.exact_bp(stack, caches, deltas)
    for i in range(L + 1):
        np.testing.assert_allclose(g[i].reshape(-1), O.path_sum(flat, J, K, i, L), rtol=1e-6, atol=1e-8)


def test_plain_mlp_analytic_jacobian_path_sum_tight():
    # J = W2 diag(phi'(W1 x)) W1 written out densely: no finite differences.
    L, d, h = 6, 3, 4
    stack = tiny_stack("mlp", L=L, d=d, h=h)
    xs, caches = O.forward(stack, RNG.normal(size=(1, d)))
    deltas = random_deltas(xs)
    J, K = [None], [None]
    for l in range(L):
        W1, W2 = stack.steps[l].W1, stack.steps[l].W2
        z = W1 @ xs[l][0]
        J.append(W2 @ np.diag(O.gelu_prime(z)) @ W1)
        K.append(np.diag(stack.gate(l)))
    flat = [x.reshape(-1) for x in deltas]
    for k in (0, 1, 2, 3, 6):
        w = O.highway_bp(stack, caches, deltas, k)
        for i in range(L + 1):
            np.testing.assert_allclose(w[i][0], O.path_sum(flat, J, K, i, k), rtol=1e-12, atol=1e-13)


def test_increment_is_paths_with_exactly_k_blocks():
    L = 4
    stack = tiny_stack("mlp", L=L)
    xs, caches = O.forward(stack, RNG.normal(size=(1, 3)))
    deltas = random_deltas(xs)
    J, K = dense_jacobians(stack, xs)
    flat = [x.reshape(-1) for x in deltas]
    hist = O.highway_bp(stack, caches, deltas, L, return_all=True)
    for k in range(1, L + 1):
        inc = hist[k][0].reshape(-1) - hist[k - 1][0].reshape(-1)
        ref = O.path_sum(flat, J, K, 0, k) - O.path_sum(flat, J, K, 0, k - 1)
        np.testing.assert_allclose(inc, ref, rtol=1e-6, atol=1e-8)


# ------------------------------------------- 2. finite differences of the loss
def _loss_from(stack, l0, x_l0, targets, coefs):
    """sum_l coefs[l] * <x_l, targets[l]> for l >= l0, running forward from x_l0."""
    x, total = x_l0, 0.0
    if coefs[l0]:
        total += float((x * targets[l0]).sum())
    for l in range(l0, stack.L):
        x = stack.gate(l) * x + stack.steps[l].forward(x)[0]
        total += float((x * targets[l + 1]).sum())
    return total


@pytest.mark.parametrize("kind", ["mlp", "preln_mlp", "rnn", "attn"])
def test_exact_bp_matches_finite_differences_of_loss(kind):
    rng = np.random.default_rng(11)
    if kind == "attn":
        d, H, S = 4, 2, 3
        Ws = [rng.normal(size=(d, d)) * 0.7 for _ in range(8)]
        steps = [O.AttnStep(*Ws[0:4], H), O.MLPStep(rng.normal(size=(6, d)), rng.normal(size=(d, 6)), True),
                 O.AttnStep(*Ws[4:8], H)]
        stack = O.Stack(steps)
        x0 = rng.normal(size=(2, S, d))
    else:
        stack = tiny_stack(kind, L=4, rng=rng)
        x0 = rng.normal(size=(2, 3))
    xs, caches = O.forward(stack, x0)
    # linear loss: L_l(x_l) = <x_l, t_l>, so delta_l = t_l exactly
    targets = [rng.normal(size=x.shape) for x in xs]
    g = O.exact_bp(stack, caches, targets)
    eps = 1e-6
    for l0 in range(stack.L + 1):
        num = np.zeros(xs[l0].size)
        for j in range(xs[l0].size):
            e = np.zeros(xs[l0].size)
            e[j] = eps
            e = e.reshape(xs[l0].shape)
            num[j] = (_loss_from(stack, l0, xs[l0] + e, targets, [1] * (stack.L + 1))
                      - _loss_from(stack, l0, xs[l0] - e, targets, [1] * (stack.L + 1))) / (2 * eps)
        np.testing.assert_allclose(g[l0].reshape(-1), num, rtol=2e-6, atol=2e-8)


def test_param_grads_match_finite_differences():
    rng = np.random.default_rng(12)
    d, H, S, h = 4, 2, 3, 6
    Wq, Wk, Wv, Wo = (rng.normal(size=(2, d, d)) * 0.6 for _ in range(4))
    W1, W2 = rng.normal(size=(2, h, d)) * 0.6, rng.normal(size=(2, d, h)) * 0.6
    params = dict(Wq=Wq, Wk=Wk, Wv=Wv, Wo=Wo, W1=W1, W2=W2)
    x0 = rng.normal(size=(2, S, d))

    def loss(p):
        st = O.transformer_stack(p["Wq"], p["Wk"], p["Wv"], p["Wo"], p["W1"], p["W2"], H)
        xs, _ = O.forward(st, x0)
        return 0.5 * float((xs[-1] ** 2).sum())

    st = O.transformer_stack(Wq, Wk, Wv, Wo, W1, W2, H)
    xs, caches = O.forward(st, x0)
    deltas = [np.zeros_like(x) for x in xs]
    deltas[-1] = xs[-1]
    g = O.exact_bp(st, caches, deltas)
    grads = O.param_grads(st, caches, xs, g, [("", l // 2) for l in range(4)])
    eps = 1e-6
    for name in params:
        assert grads[name].shape == params[name].shape
        for idx in [(0, 0, 1), (1, 2, 3), (1, 3, 0), (0, 1, 2)]:
            p2 = {k: v.copy() for k, v in params.items()}
            p2[name][idx] += eps
            up = loss(p2)
            p2[name][idx] -= 2 * eps
            dn = loss(p2)
            assert abs(grads[name][idx] - (up - dn) / (2 * eps)) < 1e-6 * max(1.0, abs(grads[name][idx]))


def test_rnn_param_and_gate_grads_match_finite_differences():
    rng = np.random.default_rng(13)
    d, nin, T, B = 3, 2, 5, 2
    W, U, a = rng.normal(size=(d, d)) * 0.5, rng.normal(size=(d, nin)), rng.uniform(0.8, 1.0, size=d)
    X, Y = rng.normal(size=(T, B, nin)), rng.normal(size=(T, B, d))
    h0 = rng.normal(size=(B, d))

    def loss(W, U, a):
        xs, _ = O.forward(O.rnn_stack(W, U, a, X), h0)
        return sum(0.5 * float(((xs[t] - Y[t - 1]) ** 2).sum()) for t in range(1, T + 1))

    st = O.rnn_stack(W, U, a, X)
    xs, caches = O.forward(st, h0)
    deltas = [np.zeros_like(h0)] + [xs[t] - Y[t - 1] for t in range(1, T + 1)]
    g = O.exact_bp(st, caches, deltas)
    grads = O.param_grads(st, caches, xs, g, [("", None)] * T)
    eps = 1e-6
    for name, P in (("W", W), ("U", U), ("a", a)):
        for idx in np.ndindex(P.shape):
            args = dict(W=W.copy(), U=U.copy(), a=a.copy())
            args[name][idx] += eps
            up = loss(**args)
            args[name][idx] -= 2 * eps
            dn = loss(**args)
            assert abs(grads[name][idx] - (up - dn) / (2 * eps)) < 2e-6 * max(1.0, abs(grads[name][idx]))


# -------------------------------- 3. exact after enough iterations (Thm 2)
@pytest.mark.parametrize("kind", ["mlp", "preln_mlp", "rnn"])
def test_exact_for_k_at_least_L_minus_i(kind):
    L = 6
    stack = tiny_stack(kind, L=L)
    xs, caches = O.forward(stack, RNG.normal(size=(3, 3)))
    deltas = random_deltas(xs)
    g = O.exact_bp(stack, caches, deltas)
    for k in range(L + 3):
        w = O.highway_bp(stack, caches, deltas, k)
        for i in range(L + 1):
            if k >= L - i:
                np.testing.assert_allclose(w[i], g[i], rtol=1e-11, atol=1e-12)
        if 0 < k < L:  # and genuinely approximate before that
            assert np.abs(w[0] - g[0]).max() > 1e-9


# ---------------------------------------------- 4. k = 0 (Eq. 5)
def test_k0_is_pure_residual_product():
    L, d = 5, 4
    stack = tiny_stack("mlp", L=L, d=d)
    xs, caches = O.forward(stack, RNG.normal(size=(2, d)))
    deltas = random_deltas(xs)
    w0 = O.highway_bp(stack, caches, deltas, 0)
    for l in range(L + 1):
        ref = np.zeros_like(xs[0])
        for j in range(l, L + 1):
            prod = np.ones(d)
            for m in range(l, j):
                prod = prod * stack.gate(m)
            ref += deltas[j] * prod
        np.testing.assert_allclose(w0[l], ref, rtol=1e-13)
    # a = 1 and a loss on the last state only: every layer sees delta_L (Section 5.1.2)
    stack1 = tiny_stack("mlp", L=L, d=d, gate="one")
    xs, caches = O.forward(stack1, RNG.normal(size=(2, d)))
    deltas = random_deltas(xs, every=False)
    for w in O.highway_bp(stack1, caches, deltas, 0):
        np.testing.assert_array_equal(w, deltas[L])


# ---------------------------------------------- 5. closed form (golden)
def test_scalar_chain_closed_form_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "scalar_chain.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 10
    for L, a, c, k, want in rows:
        L, k, a, c, want = int(L), int(k), float(a), float(c), float(want)
        stack = O.Stack([LinearStep([[c]]) for _ in range(L)], [a] * L)
        xs, caches = O.forward(stack, np.ones((1, 1)))
        deltas = [np.zeros((1, 1)) for _ in range(L)] + [np.ones((1, 1))]
        w = O.highway_bp(stack, caches, deltas, k)
        assert w[0][0, 0] == pytest.approx(want, rel=1e-13)
        binom = sum(math.comb(L, m) * c ** m * a ** (L - m) for m in range(k + 1))
        assert w[0][0, 0] == pytest.approx(binom, rel=1e-13)
        assert O.exact_bp(stack, caches, deltas)[0][0, 0] == pytest.approx((a + c) ** L, rel=1e-13)


# ---------------------------------------------- 6. special cases
def test_zero_gate_is_fixed_point_iteration():
    # K = 0: w^k_l = sum_{j=l}^{min(l+k, L)} delta_j J_j ... J_{l+1} (Section 5.2.1)
    L = 5
    stack = tiny_stack("mlp", L=L, gate="zero")
    xs, caches = O.forward(stack, RNG.normal(size=(1, 3)))
    deltas = random_deltas(xs)
    J, _ = dense_jacobians(stack, xs)
    for k in range(L + 1):
        w = O.highway_bp(stack, caches, deltas, k)
        for l in range(L + 1):
            ref = np.zeros(3)
            for j in range(l, min(l + k, L) + 1):
                vec = deltas[j].reshape(-1)
                for m in range(j, l, -1):
                    vec = vec @ J[m]
                ref = ref + vec
            np.testing.assert_allclose(w[l].reshape(-1), ref, rtol=1e-6, atol=1e-9)


def test_dead_blocks_leave_initial_estimate():
    L, d, h = 4, 3, 5
    steps = [O.MLPStep(RNG.normal(size=(h, d)), np.zeros((d, h)), True) for _ in range(L)]
    stack = O.Stack(steps, [RNG.uniform(0.5, 1.0, size=d) for _ in range(L)])
    xs, caches = O.forward(stack, RNG.normal(size=(2, d)))
    deltas = random_deltas(xs)
    w0 = O.initial_estimate(stack, deltas)
    for k in (1, 3):
        for a, b in zip(O.highway_bp(stack, caches, deltas, k), w0):
            np.testing.assert_array_equal(a, b)


# ---------------------------------------------- 7. CumSumProd (Eq. 9, 12, Alg. 1)
@pytest.mark.parametrize("n", [1, 2, 3, 7, 8, 13, 33])
def test_cumsumprod_three_ways_diagonal(n):
    rng = np.random.default_rng(100 + n)
    v = [rng.normal(size=(2, 4)) for _ in range(n)]
    gates = [rng.uniform(-1.2, 1.2, size=4) for _ in range(n)]
    seq = O.cumsumprod_sequential(v, gates)
    dfn = O.cumsumprod_definition(v, gates)
    par = O.cumsumprod_parallel(v, gates)
    for a, b, c in zip(seq, dfn, par):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(c, b, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("n", [2, 5, 6, 9])
def test_cumsumprod_parallel_dense_noncommuting(n):
    # Dense K_i of varying shape pin the order of the products and the
    # reading P_i^(0) = K_{i+1}: any other order or offset fails to type-check
    # or gives a different sum.
    rng = np.random.default_rng(200 + n)
    dims = [int(rng.integers(2, 5)) for _ in range(n)]
    v = [rng.normal(size=(dims[i],)) for i in range(n)]
    K = [rng.normal(size=(dims[i + 1], dims[i])) for i in range(n - 1)] + [None]
    par = O.cumsumprod_parallel(v, K)
    for i in range(n):
        ref = np.zeros(dims[i])
        for j in range(i, n):
            vec = v[j]
            for m in range(j - 1, i - 1, -1):
                vec = vec @ K[m]
            ref = ref + vec
        np.testing.assert_allclose(par[i], ref, rtol=1e-11, atol=1e-12)


def test_cumsumprod_textbook_cases():
    rng = np.random.default_rng(5)
    v = rng.normal(size=(11, 3))
    ones = [1.0] * 11
    ref = np.cumsum(v[::-1], axis=0)[::-1]          # identity K: reverse cumulative sum
    np.testing.assert_allclose(np.stack(O.cumsumprod_sequential(list(v), ones)), ref, rtol=1e-13)
    np.testing.assert_allclose(np.stack(O.cumsumprod_parallel(list(v), ones)), ref, rtol=1e-13)
    a, c, n = 0.9, 2.5, 20                            # constant v and K: geometric series
    out = O.cumsumprod_sequential([np.array([c])] * n, [a] * n)
    for i in range(n):
        assert out[i][0] == pytest.approx(c * (1 - a ** (n - i)) / (1 - a), rel=1e-12)


# ---------------------------------------------- 8. linearity and the folded scan
def test_linear_in_delta_and_fold_equality():
    L = 5
    stack = tiny_stack("preln_mlp", L=L)
    xs, caches = O.forward(stack, RNG.normal(size=(2, 3)))
    d1, d2 = random_deltas(xs), random_deltas(xs)
    for k in (0, 2, 5):
        w1 = O.highway_bp(stack, caches, d1, k)
        w2 = O.highway_bp(stack, caches, d2, k)
        w12 = O.highway_bp(stack, caches, [2.0 * a - 3.0 * b for a, b in zip(d1, d2)], k)
        wf = O.highway_bp_folded(stack, caches, d1, k)
        for l in range(L + 1):
            np.testing.assert_allclose(w12[l], 2.0 * w1[l] - 3.0 * w2[l], rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(wf[l], w1[l], rtol=1e-12, atol=1e-13)


# ---------------------------------------------- 9. a library's autograd
def test_exact_bp_and_param_grads_match_torch_autograd():
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F
    rng = np.random.default_rng(21)
    d, H, S, h, B, Lb = 8, 2, 5, 12, 2, 2
    P = {n: rng.normal(size=(Lb, d, d)) * 0.4 for n in ("Wq", "Wk", "Wv", "Wo")}
    P["W1"], P["W2"] = rng.normal(size=(Lb, h, d)) * 0.4, rng.normal(size=(Lb, d, h)) * 0.4
    x0 = rng.normal(size=(B, S, d))
    st = O.transformer_stack(P["Wq"], P["Wk"], P["Wv"], P["Wo"], P["W1"], P["W2"], H)
    xs, caches = O.forward(st, x0)
    deltas = [np.zeros_like(x) for x in xs]
    deltas[-1] = xs[-1]
    g = O.exact_bp(st, caches, deltas)
    grads = O.param_grads(st, caches, xs, g, [("", l // 2) for l in range(2 * Lb)])

    T = {n: torch.tensor(v, dtype=torch.float64, requires_grad=True) for n, v in P.items()}
    states = [torch.tensor(x0, dtype=torch.float64, requires_grad=True)]
    for b in range(Lb):
        x = states[-1]
        y = F.layer_norm(x, (d,), eps=1e-5)
        q, k, v = (F.linear(y, T[n][b]).view(B, S, H, d // H).transpose(1, 2) for n in ("Wq", "Wk", "Wv"))
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(1, 2).reshape(B, S, d)
        x = x + F.linear(o, T["Wo"][b])
        x.retain_grad()
        states.append(x)
        y = F.layer_norm(x, (d,), eps=1e-5)
        x = x + F.linear(F.gelu(F.linear(y, T["W1"][b])), T["W2"][b])
        x.retain_grad()
        states.append(x)
    (0.5 * (states[-1] ** 2).sum()).backward()
    for l in range(2 * Lb + 1):
        np.testing.assert_allclose(xs[l], states[l].detach().numpy(), rtol=1e-10, atol=1e-11)
        np.testing.assert_allclose(g[l], states[l].grad.numpy(), rtol=1e-9, atol=1e-11)
    for n in P:
        np.testing.assert_allclose(grads[n], T[n].grad.numpy(), rtol=1e-9, atol=1e-11)


def test_gelu_and_layernorm_pieces():
    z = np.linspace(-6, 6, 41)
    num = (O.gelu(z + 1e-6) - O.gelu(z - 1e-6)) / 2e-6
    np.testing.assert_allclose(O.gelu_prime(z), num, rtol=1e-7, atol=1e-9)
    assert O.gelu(0.0) == 0.0 and O.gelu_prime(0.0) == 0.5
    assert O.gelu(1.0) == pytest.approx(0.8413447460685429, rel=1e-14)   # Phi(1)
    x = RNG.normal(size=(3, 16)) * 3 + 1
    xhat, rstd = O.layernorm(x, 1e-5)
    np.testing.assert_allclose(xhat.mean(-1), 0, atol=1e-14)
    np.testing.assert_allclose((xhat ** 2).mean(-1), 1 - 1e-5 * rstd[:, 0] ** 2, rtol=1e-12)


# ---------------------------------------------- 10. gamma-shifted split (Appendix C.3)
def test_gamma_shift_leaves_the_network_and_exact_bp_unchanged():
    rng = np.random.default_rng(31)
    L, d = 5, 4
    base = tiny_stack("preln_mlp", L=L, d=d, gate="one", rng=rng)
    x0 = rng.normal(size=(2, d))
    xs0, c0 = O.forward(base, x0)
    deltas = random_deltas(xs0, every=False, rng=rng)
    g0 = O.exact_bp(base, c0, deltas)
    for gamma in (0.0, 0.2, 0.8, 1.0):
        st = O.shifted_stack(base, gamma)
        xs, c = O.forward(st, x0)
        for a, b in zip(xs, xs0):
            np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-14)
        for a, b in zip(O.exact_bp(st, c, deltas), g0):       # Eq. 16 and Eq. 17 agree under backpropagation
            np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
        w = O.highway_bp(st, c, deltas, L)                     # and Highway-BP still ends at the exact gradient
        for a, b in zip(w, g0):
            np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    for k in (0, 1, 3):                                        # gamma = 0 is the plain split
        for a, b in zip(O.highway_bp(O.shifted_stack(base, 0.0), c0, deltas, k), O.highway_bp(base, c0, deltas, k)):
            np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-14)


def test_gamma_one_is_fixed_point_iteration_and_path_sums_hold():
    rng = np.random.default_rng(32)
    L, d = 4, 3
    base = tiny_stack("mlp", L=L, d=d, gate="one", rng=rng)
    x0 = rng.normal(size=(1, d))
    xs, _ = O.forward(base, x0)
    deltas = random_deltas(xs, every=True, rng=rng)
    J, _ = dense_jacobians(base, xs)                            # block Jacobians by finite differences
    flat = [x.reshape(-1) for x in deltas]
    for gamma in (0.3, 1.0):
        st = O.shifted_stack(base, gamma)
        _, caches = O.forward(st, x0)
        Jg = [None] + [J[m] + gamma * np.eye(d) for m in range(1, L + 1)]
        Kg = [None] + [(1.0 - gamma) * np.eye(d)] * L
        for k in range(L + 1):
            w = O.highway_bp(st, caches, deltas, k)
            for i in range(L + 1):
                np.testing.assert_allclose(w[i].reshape(-1), O.path_sum(flat, Jg, Kg, i, k), rtol=1e-6, atol=1e-8)
    # gamma = 1: K = 0, every iteration is one more step of plain backpropagation from each loss (Section 5.2.1)
    st = O.shifted_stack(base, 1.0)
    _, caches = O.forward(st, x0)
    full = [None] + [J[m] + np.eye(d) for m in range(1, L + 1)]
    for k in range(L + 1):
        w = O.highway_bp(st, caches, deltas, k)
        for l in range(L + 1):
            ref = np.zeros(d)
            for j in range(l, min(l + k, L) + 1):
                vec = flat[j]
                for m in range(j, l, -1):
                    vec = vec @ full[m]
                ref = ref + vec
            np.testing.assert_allclose(w[l].reshape(-1), ref, rtol=1e-6, atol=1e-8)


# ---------------------------------------------- 11. GRU: a data-dependent gate (Table 1)
def _gru_setup(rng, T=4, d=3, nin=2, B=1):
    W = rng.normal(size=(3 * d, d)) * 0.7
    U = rng.normal(size=(3 * d, nin)) * 0.7
    X = rng.normal(size=(T, B, nin))
    return W, U, X, O.gru_stack(W, U, X)


def test_gru_matches_the_textbook_cell_and_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(41)
    T, d, nin, B = 5, 4, 3, 2
    W, U, X, st = _gru_setup(rng, T, d, nin, B)
    h0 = rng.normal(size=(B, d))
    xs, caches = O.forward(st, h0)
    cell = torch.nn.GRUCell(nin, d, bias=False).double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.tensor(U))
        cell.weight_hh.copy_(torch.tensor(W))
    h = torch.tensor(h0, requires_grad=True)
    hs = [h]
    for t in range(T):
        hs.append(cell(torch.tensor(X[t]), hs[-1]))
        hs[-1].retain_grad()
    # torch: h' = (1 - z) * n + z * h with the same r, z, n: the library cell is the pin for the forward map
    for t in range(T + 1):
        np.testing.assert_allclose(xs[t], hs[t].detach().numpy(), rtol=1e-12, atol=1e-13)
    Y = rng.normal(size=(T, B, d))
    loss = sum(0.5 * ((hs[t] - torch.tensor(Y[t - 1])) ** 2).sum() for t in range(1, T + 1))
    loss.backward()
    deltas = [np.zeros_like(h0)] + [xs[t] - Y[t - 1] for t in range(1, T + 1)]
    g = O.exact_bp(st, caches, deltas)
    np.testing.assert_allclose(g[0], h.grad.numpy(), rtol=1e-10, atol=1e-12)
    grads = O.param_grads(st, caches, xs, g, [("", None)] * T)
    np.testing.assert_allclose(grads["W"], cell.weight_hh.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(grads["U"], cell.weight_ih.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_gru_path_sums_with_state_dependent_gate():
    rng = np.random.default_rng(42)
    T, d = 4, 3
    W, U, X, st = _gru_setup(rng, T, d)
    xs, caches = O.forward(st, rng.normal(size=(1, d)))
    deltas = random_deltas(xs, every=True, rng=rng)
    # K_m = diag(z) from the forward pass; J_m = (Jacobian of the whole cell, by finite differences) - K_m
    J, K = [None], [None]
    for l in range(T):
        def cell(hflat, l=l):
            f, c = st.steps[l].forward(hflat.reshape(1, d))
            return (c["z"] * hflat.reshape(1, d) + f).reshape(-1)
        full = O.finite_difference_jacobian(cell, xs[l].reshape(-1), h=1e-5)
        Km = np.diag(caches[l]["z"].reshape(-1))
        K.append(Km)
        J.append(full - Km)
    flat = [x.reshape(-1) for x in deltas]
    for k in range(T + 1):
        w = O.highway_bp(st, caches, deltas, k)
        for i in range(T + 1):
            np.testing.assert_allclose(w[i].reshape(-1), O.path_sum(flat, J, K, i, k), rtol=1e-6, atol=1e-8)
    g = O.exact_bp(st, caches, deltas)
    for a, b in zip(O.highway_bp(st, caches, deltas, T), g):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    for a, b in zip(O.highway_bp_folded(st, caches, deltas, 2), O.highway_bp(st, caches, deltas, 2)):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


# ---------------------------------------------- 12. agreement sums (Figure 5)
def test_agreement_sums_on_known_vectors():
    a = np.array([3.0, 0.0, 4.0])
    b = np.array([0.0, 2.0, 4.0])
    s = O.agreement(a, b)
    np.testing.assert_allclose(s, [16.0, 25.0, 20.0, 13.0])
    # the polarisation identity ties the four together; identical inputs give cosine 1 and step 0
    assert abs(s[3] - (s[1] + s[2] - 2 * s[0])) < 1e-12
    t = O.agreement(a, a)
    assert t[0] == t[1] == t[2] and t[3] == 0.0


# ---------------------------------------------- 13. LSTM: state [c, h], gate on the cell state only (Table 1)
def test_lstm_matches_the_library_cell_and_autograd():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(51)
    T, u, nin, B = 5, 4, 3, 2
    W = rng.normal(size=(4 * u, u)) * 0.6
    U = rng.normal(size=(4 * u, nin)) * 0.6
    X = rng.normal(size=(T, B, nin))
    st = O.lstm_stack(W, U, X)
    x0 = rng.normal(size=(B, 2 * u))
    xs, caches = O.forward(st, x0)
    cell = torch.nn.LSTMCell(nin, u, bias=False).double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.tensor(U))
        cell.weight_hh.copy_(torch.tensor(W))
    x0t = torch.tensor(x0, requires_grad=True)
    c, h = x0t[:, :u], x0t[:, u:]
    states = []
    for t in range(T):
        h, c = cell(torch.tensor(X[t]), (h, c))
        states.append(torch.cat([c, h], dim=1))
    for t in range(T):
        np.testing.assert_allclose(xs[t + 1], states[t].detach().numpy(), rtol=1e-12, atol=1e-13)
    Y = rng.normal(size=(T, B, 2 * u))
    loss = sum(0.5 * ((states[t] - torch.tensor(Y[t])) ** 2).sum() for t in range(T))
    loss.backward()
    deltas = [np.zeros_like(x0)] + [xs[t + 1] - Y[t] for t in range(T)]
    g = O.exact_bp(st, caches, deltas)
    np.testing.assert_allclose(g[0], x0t.grad.numpy(), rtol=1e-10, atol=1e-12)
    grads = O.param_grads(st, caches, xs, g, [("", None)] * T)
    np.testing.assert_allclose(grads["W"], cell.weight_hh.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(grads["U"], cell.weight_ih.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_lstm_path_sums_and_exactness():
    rng = np.random.default_rng(52)
    T, u = 4, 2
    W = rng.normal(size=(4 * u, u)) * 0.7
    U = rng.normal(size=(4 * u, 2)) * 0.7
    X = rng.normal(size=(T, 1, 2))
    st = O.lstm_stack(W, U, X)
    xs, caches = O.forward(st, rng.normal(size=(1, 2 * u)))
    deltas = random_deltas(xs, every=True, rng=rng)
    J, K = [None], [None]
    for l in range(T):
        def cell(xflat, l=l):
            blk, c = st.steps[l].forward(xflat.reshape(1, 2 * u))
            return (st.steps[l].gate(c) * xflat.reshape(1, 2 * u) + blk).reshape(-1)
        full = O.finite_difference_jacobian(cell, xs[l].reshape(-1), h=1e-5)
        Km = np.diag(st.steps[l].gate(caches[l]).reshape(-1))
        K.append(Km)
        J.append(full - Km)
    flat = [x.reshape(-1) for x in deltas]
    for k in range(T + 1):
        w = O.highway_bp(st, caches, deltas, k)
        for i in range(T + 1):
            np.testing.assert_allclose(w[i].reshape(-1), O.path_sum(flat, J, K, i, k), rtol=1e-6, atol=1e-8)
    g = O.exact_bp(st, caches, deltas)
    for a, b in zip(O.highway_bp(st, caches, deltas, T), g):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


# ---------------------------------------------- 14. ReLU(x + Block(x)): a 0/1 gate that depends on the state (Table 1)
def test_relu_residual_matches_autograd_and_path_sums():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(61)
    L, d, h, N = 4, 3, 5, 2
    W1 = rng.normal(size=(L, h, d)) * 0.8
    W2 = rng.normal(size=(L, d, h)) * 0.8
    st = O.relu_mlp_stack(W1, W2)
    x0 = rng.normal(size=(N, d))
    xs, caches = O.forward(st, x0)
    # the plain definition with the library's ops
    xt = torch.tensor(x0, requires_grad=True)
    x = xt
    for l in range(L):
        x = torch.relu(x + torch.nn.functional.gelu(x @ torch.tensor(W1[l]).T) @ torch.tensor(W2[l]).T)
        np.testing.assert_allclose(xs[l + 1], x.detach().numpy(), rtol=1e-12, atol=1e-13)
    assert 0.05 < np.mean([c["mask"].mean() for c in caches]) < 0.95      # both branches of the ReLU occur
    y = rng.normal(size=(N, d))
    (0.5 * ((x - torch.tensor(y)) ** 2).sum()).backward()
    deltas = [np.zeros_like(x0) for _ in range(L)] + [xs[L] - y]
    g = O.exact_bp(st, caches, deltas)
    np.testing.assert_allclose(g[0], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    for a, b in zip(O.highway_bp(st, caches, deltas, L), g):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    # path sums with K = diag(mask), J = diag(mask) J_block (J_block by finite differences of the block alone)
    one = O.relu_mlp_stack(W1, W2)
    xs1, c1 = O.forward(one, x0[:1])
    d1 = [rng.normal(size=(1, d)) for _ in range(L + 1)]
    J, K = [None], [None]
    for l in range(L):
        blk = lambda v, l=l: one.steps[l].inner.forward(v.reshape(1, d))[0].reshape(-1)
        Jb = O.finite_difference_jacobian(blk, xs1[l].reshape(-1), h=1e-5)
        M = np.diag(c1[l]["mask"].reshape(-1))
        K.append(M)
        J.append(M @ Jb)
    flat = [v.reshape(-1) for v in d1]
    for k in range(L + 1):
        w = O.highway_bp(one, c1, d1, k)
        for i in range(L + 1):
            np.testing.assert_allclose(w[i].reshape(-1), O.path_sum(flat, J, K, i, k), rtol=1e-6, atol=1e-8)


# ---------------------------------------------- 15. post-LN layers: a row-wise gate 1 / sigma (Table 1, Appendix C.3)
def test_postln_matches_autograd_and_path_sums():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(71)
    L, d, h, N, eps = 4, 5, 6, 2, 1e-5
    W1 = rng.normal(size=(L, h, d)) * 0.7
    W2 = rng.normal(size=(L, d, h)) * 0.7
    st = O.postln_mlp_stack(W1, W2, eps)
    x0 = rng.normal(size=(N, d))
    xs, caches = O.forward(st, x0)
    xt = torch.tensor(x0, requires_grad=True)
    x = xt
    for l in range(L):
        y = x + torch.nn.functional.gelu(x @ torch.tensor(W1[l]).T) @ torch.tensor(W2[l]).T
        x = torch.nn.functional.layer_norm(y, (d,), eps=eps)
        np.testing.assert_allclose(xs[l + 1], x.detach().numpy(), rtol=1e-11, atol=1e-12)
    y_t = rng.normal(size=(N, d))
    (0.5 * ((x - torch.tensor(y_t)) ** 2).sum()).backward()
    deltas = [np.zeros_like(x0) for _ in range(L)] + [xs[L] - y_t]
    g = O.exact_bp(st, caches, deltas)
    np.testing.assert_allclose(g[0], xt.grad.numpy(), rtol=1e-9, atol=1e-11)
    for a, b in zip(O.highway_bp(st, caches, deltas, L), g):
        np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)
    # path sums on one row: K = diag(rstd), J = (Jacobian of the whole layer, by finite differences) - K
    one = O.postln_mlp_stack(W1, W2, eps)
    xs1, c1 = O.forward(one, x0[:1])
    d1 = [rng.normal(size=(1, d)) for _ in range(L + 1)]
    J, K = [None], [None]
    for l in range(L):
        def layer(v, l=l):
            blk, c = one.steps[l].forward(v.reshape(1, d))
            return (one.steps[l].gate(c) * v.reshape(1, d) + blk).reshape(-1)
        full = O.finite_difference_jacobian(layer, xs1[l].reshape(-1), h=1e-5)
        Km = np.eye(d) * float(c1[l]["rstd"].reshape(-1)[0])
        K.append(Km)
        J.append(full - Km)
    flat = [v.reshape(-1) for v in d1]
    for k in range(L + 1):
        w = O.highway_bp(one, c1, d1, k)
        for i in range(L + 1):
            np.testing.assert_allclose(w[i].reshape(-1), O.path_sum(flat, J, K, i, k), rtol=1e-5, atol=1e-7)


def test_postln_shift_leaves_the_network_and_exact_bp_unchanged():
    rng = np.random.default_rng(72)
    L, d, h, N = 5, 6, 7, 3
    W1 = rng.normal(size=(L, h, d)) * 0.5
    W2 = rng.normal(size=(L, d, h)) * 0.5
    x0 = rng.normal(size=(N, d))
    base = O.postln_mlp_stack(W1, W2)
    xs0, c0 = O.forward(base, x0)
    deltas = [np.zeros_like(x0) for _ in range(L)] + [rng.normal(size=(N, d))]
    g0 = O.exact_bp(base, c0, deltas)
    for gamma in (0.3, 0.8, 1.0):
        st = O.postln_mlp_stack(W1, W2, gamma=gamma)
        xs, c = O.forward(st, x0)
        for a, b in zip(xs, xs0):
            np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
        for a, b in zip(O.exact_bp(st, c, deltas), g0):
            np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)
        for a, b in zip(O.highway_bp(st, c, deltas, L), g0):        # exact at k = L for every split
            np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-11)
        w1 = O.highway_bp(st, c, deltas, 1)
        if gamma == 1.0:   # K = 0: one iteration reaches exactly one layer back (the fixed-point iteration)
            assert all(np.all(w1[l] == 0.0) for l in range(L - 1))
    # the shift changes the truncated estimates
    a = O.highway_bp(O.postln_mlp_stack(W1, W2, gamma=0.8), c0, deltas, 2)[0]
    b = O.highway_bp(base, c0, deltas, 2)[0]
    assert np.linalg.norm(a - b) > 1e-3 * np.linalg.norm(b)
