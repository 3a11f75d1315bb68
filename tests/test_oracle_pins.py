"""Pins for the fp64 oracle: every check here compares the oracle with
something fixed by the paper or by mathematics and computed by another route
(exact rational arithmetic, LAPACK SVD, closed forms, invariants)."""

import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import prm_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split()
            out[k] = float(v)
    return out


def _orth(n, rng):
    q, r = np.linalg.qr(rng.standard_normal((n, n)))
    return q * np.sign(np.diag(r))


def _phi5_exact(x: Fraction, iters=5) -> Fraction:
    """Scalar quintic iterate in exact rational arithmetic, coefficients as
    decimal fractions typed from the paper's hyper-parameter appendix."""
    a, b, c = Fraction(34445, 10000), Fraction(-47750, 10000), Fraction(20315, 10000)
    for _ in range(iters):
        x = a * x + b * x ** 3 + c * x ** 5
    return x


# ---------------------------------------------------------------- constants
def test_constants_match_paper():
    g = _golden()
    assert O.NS_ITERS == int(g["ns_iters"])
    assert (O.NS_A, O.NS_B, O.NS_C) == (g["ns_a"], g["ns_b"], g["ns_c"])
    cfg = O.OracleConfig()
    assert cfg.beta == g["beta"] and cfg.wd == g["wd"]
    assert cfg.gamma == g["gamma"] and cfg.K == int(g["K"])


# ------------------------------------------------------------------ NS5 pins
@pytest.mark.parametrize("sigma", [(3, 4), (1, 2, 2), (2, 3, 6), (4, 4, 7), (2, 4, 5, 6), (1, 2, 4, 10)])
@pytest.mark.parametrize("extra_cols", [0, 3])
def test_ns5_diagonal_is_scalar_quintic(sigma, extra_cols):
    # X = [diag(sigma) 0]: singular values are sigma, ||X||_F = ||sigma||_2
    # (an integer for these tuples), so NS5 acts as the scalar quintic on
    # sigma/||sigma||, which is computed exactly with rationals.
    r = len(sigma)
    nrm = math.isqrt(sum(s * s for s in sigma))
    assert nrm * nrm == sum(s * s for s in sigma)
    X = np.zeros((r, r + extra_cols))
    X[np.arange(r), np.arange(r)] = sigma
    Y = O.ns5(X, eps_ns=0.0)
    want = [float(_phi5_exact(Fraction(s, nrm))) for s in sigma]
    np.testing.assert_allclose(np.diag(Y[:, :r]), want, rtol=1e-12)
    off = Y.copy()
    off[np.arange(r), np.arange(r)] = 0.0
    assert np.all(off == 0.0)


def test_ns5_single_iteration_coefficient_placement():
    # One iteration on x*[1 0] must give a*x + b*x^3 + c*x^5 (catches a swap
    # of b and c or a wrong power).
    x = Fraction(1, 2)
    X = np.array([[3.0, 4.0]])     # norm 5 -> normalised row (0.6, 0.8), s.v. 1
    Y = O.ns5(X, eps_ns=0.0, iters=1)
    want = float(_phi5_exact(Fraction(1), iters=1))
    np.testing.assert_allclose(Y, want * np.array([[0.6, 0.8]]), rtol=1e-14)
    X = np.diag([1.0, 1.0, 1.0, 1.0])   # norm 2 -> s.v. 1/2 each
    Y = O.ns5(X, eps_ns=0.0, iters=1)
    np.testing.assert_allclose(np.diag(Y), float(_phi5_exact(x, iters=1)), rtol=1e-14)


@pytest.mark.parametrize("shape", [(2, 3), (3, 3), (4, 7), (6, 9), (16, 40)])
def test_ns5_matches_lapack_svd(shape):
    # NS5 is an odd matrix polynomial: with X = P diag(s) Q^T (LAPACK SVD),
    # NS5(X) = P diag(phi^5(s/||s||)) Q^T.
    rng = np.random.default_rng(1234 + shape[0] * 100 + shape[1])
    X = rng.standard_normal(shape)
    P, s, Qt = np.linalg.svd(X, full_matrices=False)
    x = s / np.linalg.norm(s)
    for _ in range(5):
        x = np.array([float(_phi5_exact(Fraction(v), iters=1)) for v in x])
    want = (P * x) @ Qt
    got = O.ns5(X, eps_ns=0.0)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)


def test_ns5_orthogonal_equivariance_and_transpose():
    rng = np.random.default_rng(7)
    r, c = 5, 11
    X = rng.standard_normal((r, c))
    P, Q = _orth(r, rng), _orth(c, rng)
    lhs = O.ns5(P @ X @ Q.T, 0.0)
    rhs = P @ O.ns5(X, 0.0) @ Q.T
    np.testing.assert_allclose(lhs, rhs, atol=1e-11)
    # right-handed form equals the transpose of the left-handed one
    Xn = X.T / np.linalg.norm(X)
    Y = Xn
    for _ in range(5):
        A = Y.T @ Y
        Y = O.NS_A * Y + Y @ (O.NS_B * A + O.NS_C * A @ A)
    np.testing.assert_allclose(Y.T, O.ns5(X, 0.0), atol=1e-11)


def test_ns5_scale_invariance_and_eps():
    rng = np.random.default_rng(8)
    X = rng.standard_normal((4, 6))
    np.testing.assert_allclose(O.ns5(37.5 * X, 0.0), O.ns5(X, 0.0), atol=1e-12)
    assert np.all(O.ns5(np.zeros((3, 5)), 1e-7) == 0.0)
    # eps_ns enters as ||X||_F + eps_ns
    Y = O.ns5(X, 0.5, iters=0)
    np.testing.assert_allclose(Y, X / (np.linalg.norm(X) + 0.5), rtol=1e-15)


def test_ns5_is_not_the_polar_factor_but_lands_near_it():
    # after 5 iterations singular values sit in a band around 1, not at 1
    rng = np.random.default_rng(9)
    X = rng.standard_normal((32, 96))
    s = np.linalg.svd(O.ns5(X, 0.0), compute_uv=False)
    assert s.min() > 0.3 and s.max() < 1.25
    assert np.abs(s - 1).max() > 1e-3


# -------------------------------------------------------------- RowNorm pins
def test_rownorm_unit_rows_and_inner_product_identity():
    rng = np.random.default_rng(11)
    X = rng.standard_normal((7, 13)) * np.exp(rng.standard_normal((7, 1)))
    R = O.rownorm(X, 1e-8)
    np.testing.assert_allclose(np.linalg.norm(R, axis=1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(np.linalg.norm(R), math.sqrt(7), rtol=1e-14)
    np.testing.assert_allclose(np.sum(X * R), np.linalg.norm(X, axis=1).sum(), rtol=1e-13)
    assert np.all(np.sign(R) == np.sign(X))
    alpha = np.exp(rng.standard_normal((7, 1)))
    np.testing.assert_allclose(O.rownorm(alpha * X, 1e-8), R, rtol=1e-13)


def test_rownorm_is_the_l2inf_maximiser():
    rng = np.random.default_rng(12)
    X = rng.standard_normal((5, 9))
    best = np.sum(X * O.rownorm(X, 1e-8))
    for _ in range(200):
        V = rng.standard_normal((5, 9))
        V /= np.maximum(np.linalg.norm(V, axis=1, keepdims=True), 1.0)
        assert np.sum(X * V) <= best + 1e-12


def test_rownorm_clamp_zero_and_tiny_rows():
    X = np.array([[0.0, 0.0, 0.0], [3e-9, 4e-9, 0.0], [3.0, 4.0, 0.0]])
    R = O.rownorm(X, 1e-8)
    assert np.all(R[0] == 0.0)
    np.testing.assert_allclose(R[1], [0.3, 0.4, 0.0], rtol=1e-14)     # divided by eps
    np.testing.assert_allclose(R[2], [0.6, 0.8, 0.0], rtol=1e-14)


def test_tall_rownorm_is_column_norm_sharded_sum():
    # Tall stored matrix: RowNorm acts on the transpose, i.e. on stored
    # columns, and partial column sums over any row partition add up
    # (sharded RowNorm proposition).
    rng = np.random.default_rng(13)
    M = rng.standard_normal((12, 5))
    cfg = O.OracleConfig(gamma=1.0)
    D = O.direction(M, refresh=False, cfg=cfg)
    parts = [M[:3], M[3:4], M[4:]]
    nu = np.sqrt(sum((p * p).sum(axis=0) for p in parts))
    np.testing.assert_allclose(D, M / nu, rtol=1e-13)
    np.testing.assert_allclose(np.linalg.norm(D, axis=0), 1.0, rtol=1e-13)


def test_square_is_not_transposed():
    rng = np.random.default_rng(14)
    M = rng.standard_normal((6, 6))
    D = O.direction(M, refresh=False, cfg=O.OracleConfig(gamma=1.0))
    np.testing.assert_allclose(np.linalg.norm(D, axis=1), 1.0, rtol=1e-13)
    assert np.abs(np.linalg.norm(D, axis=0) - 1.0).max() > 1e-3
    assert O.orient(np.zeros((3, 5))).shape == (3, 5)
    assert O.orient(np.zeros((5, 3))).shape == (3, 5)
    assert O.orient_inv(np.zeros((3, 5)), 5, 3).shape == (5, 3)


# --------------------------------------------------------- momentum and step
@pytest.mark.parametrize("nesterov", [False, True])
def test_momentum_constant_gradient_closed_form(nesterov):
    # constant G from M=0: M_t = (1-beta^(t+1)) G, Nesterov U_t = (1-beta^(t+2)) G
    rng = np.random.default_rng(15)
    G = rng.standard_normal((3, 4))
    beta = 0.95
    M = np.zeros_like(G)
    for t in range(6):
        M = O.momentum_update(M, G, beta)
        np.testing.assert_allclose(M, (1 - beta ** (t + 1)) * G, rtol=1e-13)
        U = O.direction_input(M, G, beta, nesterov)
        k = (1 - beta ** (t + 2)) if nesterov else (1 - beta ** (t + 1))
        np.testing.assert_allclose(U, k * G, rtol=1e-13)


def test_schedule_and_grouping():
    assert [t for t in range(8) if O.is_refresh(t, 4)] == [0, 4]   # 2 refreshes + 6 row steps
    assert all(O.is_refresh(t, 1) for t in range(5))
    with pytest.raises(ValueError):
        O.is_refresh(0, 0)
    shapes = [(2, 6), (2, 2), (8, 2), (2, 8), (2, 6), (8, 2), (2, 2)]
    g, o, gs = O.group_by_shape(shapes)
    assert g == [0, 1, 2, 3, 0, 2, 1]
    assert o == [0, 0, 0, 0, 1, 1, 1]
    assert gs == [(2, 6), (2, 2), (8, 2), (2, 8)]


def _rand_case(rng, m, n):
    W = rng.standard_normal((m, n)) * 0.02
    G = rng.standard_normal((m, n))
    M = rng.standard_normal((m, n)) * 0.1
    return W, G, M


@pytest.mark.parametrize("shape", [(4, 9), (9, 4), (5, 5)])
def test_row_step_norm_target_sign_and_decay(shape):
    rng = np.random.default_rng(16)
    m, n = shape
    W, G, M = _rand_case(rng, m, n)
    cfg = O.OracleConfig(K=4, nesterov=True, lr=5e-3, wd=0.01, gamma=0.15)
    Wn, Mn = O.step_matrix(W, G, M, t=1, cfg=cfg)
    delta = Wn - (1 - cfg.lr * cfg.wd) * W
    s = math.sqrt(max(1.0, m / n))
    axis = 1 if m <= n else 0
    np.testing.assert_allclose(np.linalg.norm(delta, axis=axis), cfg.lr * s * cfg.gamma, rtol=1e-12)
    U = cfg.beta * Mn + (1 - cfg.beta) * G
    assert np.all(np.sign(delta) == -np.sign(U))
    # zero direction input: only the decay acts
    Wz, _ = O.step_matrix(W, np.zeros_like(G), np.zeros_like(M), t=1, cfg=cfg)
    np.testing.assert_allclose(Wz, (1 - 5e-3 * 0.01) * W, rtol=1e-15)
    # lr = 0 leaves the weights alone, momentum still moves
    cfg0 = O.OracleConfig(K=4, nesterov=True, lr=0.0)
    W0, M0 = O.step_matrix(W, G, M, t=1, cfg=cfg0)
    assert np.array_equal(W0, W) and not np.array_equal(M0, M)


@pytest.mark.parametrize("shape", [(4, 9), (9, 4)])
def test_refresh_step_uses_ns5_without_gamma(shape):
    rng = np.random.default_rng(17)
    m, n = shape
    W, G, M = _rand_case(rng, m, n)
    cfg = O.OracleConfig(K=4, nesterov=False, lr=1e-2, wd=0.0, gamma=0.15, eps_ns=0.0, scale_mode=0)
    Wn, Mn = O.step_matrix(W, G, M, t=4, cfg=cfg)
    D = (W - Wn) / cfg.lr
    # singular values of the direction equal the scalar quintic of the
    # momentum's normalised singular values (LAPACK), untouched by gamma
    Mt = 0.95 * M + 0.05 * G
    s = np.linalg.svd(Mt, compute_uv=False)
    x = s / np.linalg.norm(s)
    want = sorted(float(_phi5_exact(Fraction(v))) for v in x)
    got = sorted(np.linalg.svd(D, compute_uv=False))
    np.testing.assert_allclose(got, want, rtol=1e-9)
    # gamma must not matter on a refresh step, K=1 makes every step a refresh
    cfg2 = O.OracleConfig(K=1, nesterov=False, lr=1e-2, wd=0.0, gamma=0.9, eps_ns=0.0, scale_mode=0)
    Wn2, _ = O.step_matrix(W, G, M, t=3, cfg=cfg2)
    np.testing.assert_allclose(Wn2, Wn, rtol=1e-14)


def test_gamma_scales_row_branch_only_and_shape_scale():
    rng = np.random.default_rng(18)
    W, G, M = _rand_case(rng, 8, 2)
    base = dict(K=2, nesterov=False, lr=1e-2, wd=0.0)
    a, _ = O.step_matrix(W, G, M, 1, O.OracleConfig(gamma=0.15, **base))
    b, _ = O.step_matrix(W, G, M, 1, O.OracleConfig(gamma=0.30, **base))
    np.testing.assert_allclose(W - b, 2 * (W - a), rtol=1e-12)
    c, _ = O.step_matrix(W, G, M, 1, O.OracleConfig(gamma=0.15, scale_mode=0, **base))
    np.testing.assert_allclose(W - a, 2.0 * (W - c), rtol=1e-12)     # sqrt(8/2) = 2
    assert O.shape_scale(2, 8, 1) == 1.0 and O.shape_scale(8, 2, 1) == 2.0


def test_momentum_form_invariance():
    # accumulate-form momentum M' = beta M' + G gives the same weights
    rng = np.random.default_rng(19)
    m, n = 4, 7
    W = rng.standard_normal((m, n)) * 0.02
    cfg = O.OracleConfig(K=2, nesterov=True, lr=5e-3, wd=0.01, eps_ns=0.0, eps_row=0.0)
    W1, M1 = W.copy(), np.zeros((m, n))
    W2, M2 = W.copy(), np.zeros((m, n))
    for t in range(4):
        G = rng.standard_normal((m, n))
        W1, M1 = O.step_matrix(W1, G, M1, t, cfg)
        M2 = cfg.beta * M2 + G
        U2 = cfg.beta * M2 + G
        D2 = O.direction(U2, O.is_refresh(t, cfg.K), cfg)
        W2 = (1 - cfg.lr * cfg.wd) * W2 - cfg.lr * D2
        np.testing.assert_allclose(M2 * (1 - cfg.beta), M1, rtol=1e-12)
    np.testing.assert_allclose(W2, W1, rtol=1e-11)
