"""Pins of the CPU oracle against things that are not the oracle: a hand-worked example,
closed forms evaluated in arbitrary-precision decimal arithmetic, exact integer brute force,
special cases that reduce to library routines (numpy float64 GEMM, torch float64 layer_norm,
scipy's erf), and invariants of the operator."""
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_01884_b200 import workloads as wk

getcontext().prec = 60
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ACTS = [wk.ACT_IDENTITY, wk.ACT_RELU, wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU]


# ---- independent closed forms (decimal arithmetic, no libm) -------------------------
def _pi() -> Decimal:
    # Machin: pi = 16 atan(1/5) - 4 atan(1/239)
    def atan_inv(q):
        x = Decimal(1) / q
        s, t, n, x2 = x, x, 1, x * x
        while abs(t) > Decimal(10) ** -58:
            t = -t * x2
            n += 2
            s += t / n
        return s
    return 16 * atan_inv(Decimal(5)) - 4 * atan_inv(Decimal(239))


PI = _pi()


def d_erf(x: Decimal) -> Decimal:
    # Maclaurin series  erf x = 2/sqrt(pi) * sum (-1)^n x^(2n+1) / (n! (2n+1))
    s, term, n = Decimal(0), x, 0
    while True:
        add = term / (2 * n + 1)
        s += add
        if abs(add) < Decimal(10) ** -55:
            break
        n += 1
        term = -term * x * x / n
    return 2 * s / PI.sqrt()


def d_tanh(x: Decimal) -> Decimal:
    e = (2 * x).exp()
    return (e - 1) / (e + 1)


def d_act(kind: int, z: float) -> float:
    x = Decimal(z)
    if kind == wk.ACT_IDENTITY:
        r = x
    elif kind == wk.ACT_RELU:
        r = x if x > 0 else Decimal(0)
    elif kind == wk.ACT_GELU_ERF:
        r = x * (1 + d_erf(x / Decimal(2).sqrt())) / 2
    elif kind == wk.ACT_GELU_TANH:
        r = x * (1 + d_tanh((2 / PI).sqrt() * (x + Decimal("0.044715") * x ** 3))) / 2
    else:
        r = x / (1 + (-x).exp())
    return float(r)


POINTS = [-6.0, -3.0, -1.0, -0.5, -1e-3, 0.0, 1e-3, 0.25, 1.0, 2.0, 4.5]


@pytest.mark.parametrize("kind", ACTS)
def test_activation_matches_decimal_closed_form(kind):
    for z in POINTS:
        assert oracle.act(kind, z) == pytest.approx(d_act(kind, z), rel=1e-13, abs=1e-15)


def test_activation_textbook_values():
    # Phi(1) and Phi(2) from the standard normal table; logistic(1) = 1/(1+1/e).
    assert oracle.act(wk.ACT_GELU_ERF, 1.0) == pytest.approx(0.8413447460685429, abs=1e-15)
    assert oracle.act(wk.ACT_GELU_ERF, -1.0) == pytest.approx(-0.15865525393145707, abs=1e-15)
    assert oracle.act(wk.ACT_GELU_ERF, 2.0) == pytest.approx(2 * 0.9772498680518208, abs=1e-15)
    assert oracle.act(wk.ACT_SILU, 1.0) == pytest.approx(0.7310585786300049, abs=1e-15)
    assert oracle.act(wk.ACT_SILU, -1.0) == pytest.approx(-0.2689414213699951, abs=1e-15)
    for kind in ACTS:
        assert oracle.act(kind, 0.0) == 0.0
    assert oracle.act(wk.ACT_RELU, -2.5) == 0.0 and oracle.act(wk.ACT_RELU, 2.5) == 2.5


def test_activation_identities_and_scipy():
    from scipy.special import erf as sp_erf, expit
    for z in np.linspace(-8, 8, 161):
        z = float(z)
        for kind in (wk.ACT_GELU_ERF, wk.ACT_GELU_TANH, wk.ACT_SILU):
            # f(z) - f(-z) = z for z*s(z) with s(z)+s(-z)=1
            assert oracle.act(kind, z) - oracle.act(kind, -z) == pytest.approx(z, abs=1e-14)
        assert oracle.act(wk.ACT_GELU_ERF, z) == pytest.approx(0.5 * z * (1 + sp_erf(z / math.sqrt(2))), abs=1e-14)
        assert oracle.act(wk.ACT_SILU, z) == pytest.approx(z * expit(z), abs=1e-14)
        assert abs(oracle.act(wk.ACT_GELU_ERF, z) - oracle.act(wk.ACT_GELU_TANH, z)) < 1e-3


# ---- the hand-worked example ---------------------------------------------------------
def _golden():
    g = {}
    with open(os.path.join(GOLDEN, "worked_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            g[k] = np.array([float(t) for t in v])
    return g


def test_worked_example():
    g = _golden()
    M, N, K = int(g["M"][0]), int(g["N"][0]), int(g["K"][0])
    X, W, b = g["X"].reshape(M, K), g["W"].reshape(N, K), g["b"]
    assert np.array_equal(oracle.fused_linear(X, W, b), g["Z"].reshape(M, N))
    assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU), g["E_relu"].reshape(M, N))
    assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU, red=wk.RED_SUM), g["sum"])
    assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU, red=wk.RED_MAX), g["max"])
    one, zero = np.ones(N), np.zeros(N)
    ln = oracle.fused_linear(X, W, b, one, zero, act=wk.ACT_RELU, red=wk.RED_LAYERNORM, eps=0.0, rows=[0])
    assert ln[0] == pytest.approx(g["ln_row0_num"] / math.sqrt(g["ln_row0_den_sq"][0]), abs=1e-15)
    beta = np.array([0.25, -0.5, 2.0])
    ln = oracle.fused_linear(X, W, b, 3 * one, beta, act=wk.ACT_RELU, red=wk.RED_LAYERNORM, eps=1e-5)
    assert np.array_equal(ln[1], beta)            # constant row: exactly beta


# ---- contraction and bias --------------------------------------------------------------
@pytest.mark.parametrize("kind", ACTS)
def test_identity_weight_reproduces_activation_of_x(kind):
    rng = np.random.default_rng(1)
    X = rng.standard_normal((7, 5)).astype(np.float32) * 2
    got = oracle.fused_linear(X, np.eye(5, dtype=np.float32), None, act=kind, scale=0.5)
    want = np.array([[0.5 * d_act(kind, float(v)) for v in row] for row in X])
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("kind", ACTS)
def test_all_ones_gives_act_of_k_plus_bias(kind):
    M, N, K = 3, 6, 9
    b = np.array([-12.0, -9.5, -9.0, -8.0, 0.0, 1.5], dtype=np.float32)
    X, W = np.ones((M, K), np.float32), np.ones((N, K), np.float32)
    e = np.array([2.0 * d_act(kind, K + float(v)) for v in b])
    np.testing.assert_allclose(oracle.fused_linear(X, W, b, act=kind, scale=2.0), np.tile(e, (M, 1)), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(oracle.fused_linear(X, W, b, act=kind, scale=2.0, red=wk.RED_SUM), np.full(M, e.sum()), rtol=1e-13)
    np.testing.assert_allclose(oracle.fused_linear(X, W, b, act=kind, scale=2.0, red=wk.RED_MAX), np.full(M, e.max()), rtol=1e-13)


def test_brute_force_small_integers_exact():
    """Integer inputs: every product and sum is exact, so the oracle must equal rational
    arithmetic done a different way (column-at-a-time with Fractions)."""
    rng = np.random.default_rng(7)
    for M, N, K in [(1, 1, 1), (2, 3, 4), (5, 4, 3), (3, 5, 5), (4, 2, 1)]:
        X = rng.integers(-4, 5, (M, K)).astype(np.float32)
        W = rng.integers(-4, 5, (N, K)).astype(np.float32)
        b = rng.integers(-3, 4, N).astype(np.float32)
        Z = [[Fraction(int(b[n])) for n in range(N)] for _ in range(M)]
        for k in range(K):                       # outer-product order, not the oracle's
            for n in range(N):
                for m in range(M):
                    Z[m][n] += Fraction(int(X[m, k])) * Fraction(int(W[n, k]))
        Zf = np.array([[float(v) for v in row] for row in Z])
        assert np.array_equal(oracle.fused_linear(X, W, b), Zf)
        R = np.maximum(Zf, 0) * 3
        assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU, scale=3.0), R)
        assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU, scale=3.0, red=wk.RED_SUM), R.sum(1))
        assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_RELU, scale=3.0, red=wk.RED_MAX), R.max(1))
        assert np.array_equal(oracle.fused_linear(X, W, None), Zf - b)       # bias really optional


def test_reduces_to_library_gemm():
    rng = np.random.default_rng(3)
    M, N, K = 13, 29, 37                         # all different: a transposed operand cannot pass
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    want = X.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_allclose(oracle.fused_linear(X, W, b), want, rtol=0, atol=1e-12)


def test_scale_is_applied_after_the_activation():
    X = np.array([[1.0]], np.float32)
    W = np.array([[1.0]], np.float32)
    got = oracle.fused_linear(X, W, None, act=wk.ACT_GELU_ERF, scale=0.5)[0, 0]
    assert got == pytest.approx(0.5 * 0.8413447460685429, abs=1e-15)      # not gelu(0.5)


# ---- LayerNorm -------------------------------------------------------------------------
def _ln_case(seed=5, M=6, N=33, K=17):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) / 4).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32) * 0.1
    g = rng.uniform(0.5, 1.5, N).astype(np.float32)
    be = rng.standard_normal(N).astype(np.float32)
    return X, W, b, g, be


def test_layernorm_reduces_to_library_routine():
    import torch
    X, W, b, g, be = _ln_case()
    E = oracle.fused_linear(X, W, b, act=wk.ACT_GELU_TANH, scale=1.5)
    want = torch.nn.functional.layer_norm(torch.from_numpy(E), (E.shape[1],),
                                          torch.from_numpy(g).double(), torch.from_numpy(be).double(), 1e-5).numpy()
    got = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_GELU_TANH, scale=1.5, red=wk.RED_LAYERNORM, eps=1e-5)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def test_layernorm_invariants():
    X, W, b, g, be = _ln_case(seed=9)
    N = W.shape[0]
    one, zero = np.ones(N, np.float32), np.zeros(N, np.float32)
    eps = 1e-5
    E = oracle.fused_linear(X, W, b, act=wk.ACT_GELU_ERF)
    y = oracle.fused_linear(X, W, b, one, zero, act=wk.ACT_GELU_ERF, red=wk.RED_LAYERNORM, eps=eps)
    var = E.var(axis=1)
    assert np.abs(y.mean(1)).max() < 1e-6
    assert np.abs(y.var(1) - var / (var + eps)).max() < 1e-6
    y0 = oracle.fused_linear(X, W, b, one, zero, act=wk.ACT_GELU_ERF, red=wk.RED_LAYERNORM, eps=1e-12)
    assert np.abs(y0.var(1) - 1.0).max() < 1e-6          # unit variance once eps is negligible
    # affine part: y(gamma, beta) = gamma * y(1, 0) + beta
    ya = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_GELU_ERF, red=wk.RED_LAYERNORM, eps=eps)
    np.testing.assert_allclose(ya, y * g.astype(np.float64) + be.astype(np.float64), atol=1e-13)
    # with eps = 0 a positive scale of E drops out
    a = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_RELU, scale=1.0, red=wk.RED_LAYERNORM, eps=0.0)
    c = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_RELU, scale=8.0, red=wk.RED_LAYERNORM, eps=0.0)
    np.testing.assert_allclose(a, c, atol=1e-12)


# ---- reductions and row subsets -----------------------------------------------------------
def test_reductions_agree_with_unreduced_output():
    X, W, b, _, _ = _ln_case(seed=11, M=9, N=21, K=8)
    E = oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=0.7)
    np.testing.assert_allclose(oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=0.7, red=wk.RED_SUM), E.sum(1), rtol=1e-14)
    assert np.array_equal(oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=0.7, red=wk.RED_MAX), E.max(1))
    # all-negative row: the max must not be clamped at zero
    Xn = -np.abs(X)
    Wp = np.abs(W)
    En = oracle.fused_linear(Xn, Wp, None)
    assert (En < 0).all()
    assert np.array_equal(oracle.fused_linear(Xn, Wp, None, red=wk.RED_MAX), En.max(1))


def test_row_subset_equals_full_rows():
    wl = wk.WORKLOADS["c1"]
    i = wk.make_inputs(wl)
    full = oracle.fused_linear(i["X"], i["W"], i["b"], act=wl.act, scale=wl.scale, red=wl.red)
    rows = wk.sample_rows(wl.M, tile=16)
    sub = oracle.fused_linear(i["X"], i["W"], i["b"], act=wl.act, scale=wl.scale, red=wl.red, rows=rows)
    assert np.array_equal(sub, full[rows])
    X, W, b, g, be = _ln_case(seed=2, M=40)
    f = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_SILU, red=wk.RED_LAYERNORM)
    s = oracle.fused_linear(X, W, b, g, be, act=wk.ACT_SILU, red=wk.RED_LAYERNORM, rows=[39, 0, 17])
    assert np.array_equal(s, f[[39, 0, 17]])


def test_bad_arguments_are_rejected():
    X, W = np.ones((2, 3), np.float32), np.ones((4, 3), np.float32)
    with pytest.raises(ValueError):
        oracle.fused_linear(X, W, None, red=wk.RED_LAYERNORM)        # gamma/beta missing
    with pytest.raises(ValueError):
        oracle.fused_linear(X, W, None, rows=[2])                    # row out of range
    with pytest.raises(ValueError):
        oracle.fused_linear(X, np.ones((4, 2), np.float32))          # K mismatch


# ---- the case-study chain: Linear, subtract, row mean, GELU, residual add ---------------------
def test_chain_worked_example():
    g = _golden()
    M, N, K = int(g["M"][0]), int(g["N"][0]), int(g["K"][0])
    X, W, b = g["X"].reshape(M, K), g["W"].reshape(N, K), g["b"]
    y = oracle.fused_linear(X, W, b, red=wk.RED_MEAN_GELU_RESIDUAL, sub=g["sub"])
    assert y.shape == (M, K)
    mean = g["rowmean_num"] / g["rowmean_den"]
    want0 = X[0] + d_act(wk.ACT_GELU_ERF, float(Fraction(4, 3)))
    np.testing.assert_allclose(y[0], want0, rtol=0, atol=1e-15)
    np.testing.assert_allclose(y[1], X[1] + g["gelu_of_minus_one"][0], rtol=0, atol=1e-15)
    assert mean[1] == -1.0


def test_chain_reduces_to_a_matrix_vector_product():
    """The row mean of a linear map is linear: mean_n(X W^T + b - sub) = X wbar + mean(b - sub),
    with wbar the mean of W's rows -- a float64 library GEMV plus the decimal GELU."""
    rng = np.random.default_rng(21)
    M, N, K = 9, 14, 11
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    sub = rng.standard_normal(N).astype(np.float32)
    mu = X.astype(np.float64) @ W.astype(np.float64).mean(0) + (b.astype(np.float64) - sub.astype(np.float64)).mean()
    want = X.astype(np.float64) + np.array([d_act(wk.ACT_GELU_ERF, float(v)) for v in mu])[:, None]
    got = oracle.fused_linear(X, W, b, red=wk.RED_MEAN_GELU_RESIDUAL, sub=sub)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    # with an activation and a scale in front, the mean is taken of scale*act(Z) - sub
    E = oracle.fused_linear(X, W, b, act=wk.ACT_RELU, scale=0.5)
    mu2 = (E - sub.astype(np.float64)).mean(1)
    want2 = X.astype(np.float64) + np.array([d_act(wk.ACT_GELU_ERF, float(v)) for v in mu2])[:, None]
    got2 = oracle.fused_linear(X, W, b, act=wk.ACT_RELU, scale=0.5, red=wk.RED_MEAN_GELU_RESIDUAL, sub=sub)
    np.testing.assert_allclose(got2, want2, rtol=0, atol=1e-12)


def test_chain_special_cases():
    rng = np.random.default_rng(22)
    X = rng.standard_normal((4, 6)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    # zero weights and sub = b: the mean is exactly 0, gelu(0) = 0, the output is the input
    y = oracle.fused_linear(X, np.zeros((5, 6), np.float32), b, red=wk.RED_MEAN_GELU_RESIDUAL, sub=b)
    assert np.array_equal(y, X.astype(np.float64))
    # no subtract vector means nothing is subtracted
    W = rng.standard_normal((5, 6)).astype(np.float32)
    y0 = oracle.fused_linear(X, W, b, red=wk.RED_MEAN_GELU_RESIDUAL)
    y1 = oracle.fused_linear(X, W, b, red=wk.RED_MEAN_GELU_RESIDUAL, sub=np.zeros(5, np.float32))
    assert np.array_equal(y0, y1)
    # row subset
    ys = oracle.fused_linear(X, W, b, red=wk.RED_MEAN_GELU_RESIDUAL, rows=[3, 1])
    assert np.array_equal(ys, y0[[3, 1]])


# ---- log-sum-exp and per-row cross-entropy ---------------------------------------------------------
def test_logsumexp_closed_forms():
    # all logits equal to c: log(N e^c) = c + log N; identity weights make the logits X itself
    N = 7
    X = np.full((2, N), 1.25, np.float32)
    got = oracle.fused_linear(X, np.eye(N, dtype=np.float32), None, red=wk.RED_LOGSUMEXP)
    assert got == pytest.approx(np.full(2, 1.25 + float(Decimal(N).ln())), abs=1e-14)
    # two logits a, b: log(e^a + e^b) in decimal arithmetic
    X = np.array([[0.5, -1.5], [30.0, 29.0]], np.float32)
    got = oracle.fused_linear(X, np.eye(2, dtype=np.float32), None, red=wk.RED_LOGSUMEXP)
    want = [float((Decimal(a).exp() + Decimal(b).exp()).ln()) for a, b in X.tolist()]
    assert got == pytest.approx(want, rel=1e-14)
    # large logits must not overflow: exp(1000) is not representable, the result is
    got = oracle.fused_linear(np.array([[1000.0, 1000.0]], np.float32), np.eye(2, dtype=np.float32), None, red=wk.RED_LOGSUMEXP)
    assert got[0] == pytest.approx(1000.0 + math.log(2.0), rel=1e-15)


def test_logsumexp_and_cross_entropy_reduce_to_library_routines():
    import torch
    from scipy.special import logsumexp as sp_lse
    rng = np.random.default_rng(31)
    M, N, K = 11, 23, 9
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((N, K)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32)
    t = rng.integers(0, N, M).astype(np.int32)
    E = oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=2.0)
    lse = oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=2.0, red=wk.RED_LOGSUMEXP)
    np.testing.assert_allclose(lse, sp_lse(E, axis=1), rtol=0, atol=1e-12)
    ce = oracle.fused_linear(X, W, b, act=wk.ACT_SILU, scale=2.0, red=wk.RED_CROSS_ENTROPY, target=t)
    want = torch.nn.functional.cross_entropy(torch.from_numpy(E), torch.from_numpy(t).long(), reduction="none").numpy()
    np.testing.assert_allclose(ce, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(ce, lse - E[np.arange(M), t], rtol=0, atol=1e-13)
    # invariants: shifting every logit of a row by c shifts lse by c and leaves the loss alone
    ce2 = oracle.fused_linear(X, W, b + 3.0, red=wk.RED_CROSS_ENTROPY, target=t)
    ce1 = oracle.fused_linear(X, W, b, red=wk.RED_CROSS_ENTROPY, target=t)
    np.testing.assert_allclose(ce1, ce2, rtol=0, atol=1e-5)          # b + 3 is rounded to fp32 once
    assert (ce >= 0).all() and (lse >= E.max(1)).all()
    # row subset, and a dominant class has zero loss
    sub = oracle.fused_linear(X, W, b, red=wk.RED_CROSS_ENTROPY, target=t, rows=[10, 2])
    assert np.array_equal(sub, ce1[[10, 2]])
    Xd = np.zeros((1, 3), np.float32)
    bd = np.array([0.0, 200.0, 0.0], np.float32)
    assert oracle.fused_linear(Xd, np.zeros((3, 3), np.float32), bd, red=wk.RED_CROSS_ENTROPY, target=[1])[0] == pytest.approx(0.0, abs=1e-80)
    with pytest.raises(ValueError):
        oracle.fused_linear(X, W, b, red=wk.RED_CROSS_ENTROPY)                      # targets missing
    with pytest.raises(ValueError):
        oracle.fused_linear(X, W, b, red=wk.RED_CROSS_ENTROPY, target=np.full(M, N))  # class out of range
