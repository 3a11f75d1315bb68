"""A numpy emulation of NS5 with bf16-rounded operands and fp32 accumulation.

Test infrastructure, written for the tests alone: it shares nothing with the
CUDA sources and is not part of the oracle.  It answers one question: how far
from the exact (fp64) recurrence does the arithmetic *format* of the
tensor-core path land, whatever kernel executes it?  Every matrix that path
stores (the input X_0, every Gram matrix, every polynomial B_k, every
intermediate X_k) is rounded to bf16 (round to nearest even); every product is
accumulated in fp32.  Two orders of evaluation are emulated:

* `ns5_bf16_printed`: the recurrence as the paper prints it (Appendix
  Eq. app-ns-recurrence), five times  A = X X^T, B = bA + cA^2, X <- aX + BX.
* `ns5_bf16_gramspace`: the same polynomial with the first three iterations on
  the r x r Gram matrix (A_{k+1} = P_k A_k P_k with P_k = aI + B_k, and the
  running product of the P_k applied to X_0 once), optionally with the last
  Gram matrix taken from the one before it.

The Frobenius scale alpha = 1/(||X||_F + eps) is applied where the tensor-core
path applies it: on the first Gram matrix (alpha^2) and on the first update
(alpha), so that X_0 is rounded to bf16 before it is scaled.
"""

import numpy as np

NS_A, NS_B, NS_C = 3.4445, -4.7750, 2.0315


def bf16_round(x):
    """Round an fp32 array to the nearest bf16 value (ties to even), returned as fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_split_round(x):
    """x kept as the sum of two bf16 numbers (hi = bf16(x), lo = bf16(x - hi)): 16 mantissa bits
    instead of 8, what a product costs three (symmetric) or two tensor-core passes to consume."""
    hi = bf16_round(x)
    return hi + bf16_round(np.asarray(x, dtype=np.float32) - hi)


def _f32(x):
    return np.asarray(x, dtype=np.float32)


def ns5_fp64(U, eps_ns=1e-7):
    """The exact recurrence (fp64), written out again here so that this file
    stands alone; tests compare it with the oracle's."""
    X = np.asarray(U, dtype=np.float64)
    X = X / (np.sqrt(np.sum(X * X)) + eps_ns)
    for _ in range(5):
        A = X @ X.T
        B = NS_B * A + NS_C * (A @ A)
        X = NS_A * X + B @ X
    return X


def ns5_bf16_printed(U, eps_ns=1e-7, rnd=bf16_round, rnd_rr=None):
    """Five printed iterations, bf16 storage (rnd), fp32 accumulation.  With
    rnd = identity this is plain fp32 arithmetic.  rnd_rr, if given, is the
    storage of the r x r matrices A and B alone."""
    rnd_rr = rnd if rnd_rr is None else rnd_rr
    U = _f32(U)
    al = np.float32(1.0 / (np.sqrt(np.sum(U.astype(np.float64) ** 2)) + eps_ns))
    X = rnd(U)
    for k in range(5):
        A = X @ X.T
        if k == 0:
            A = A * (al * al)
        A = rnd_rr(A)
        B = rnd_rr(np.float32(NS_B) * A + np.float32(NS_C) * (A @ A))
        Xn = np.float32(NS_A) * X + B @ X
        if k == 0:
            Xn = al * Xn
        X = rnd(Xn) if k < 4 else Xn
    return X


def ns5_bf16_gramspace(U, last_gram_from_previous, eps_ns=1e-7, rnd=bf16_round, rnd_x0=None):
    """Iterations 1-3 on the Gram matrix, 4 and 5 as printed; with
    last_gram_from_previous the Gram matrix of iteration 5 is P_3 A_3 P_3
    instead of X_4 X_4^T.  rnd_x0, if given, is the storage of the input X_0
    alone (it enters two products: X_0 X_0^T and Q X_0)."""
    a, b, c = np.float32(NS_A), np.float32(NS_B), np.float32(NS_C)
    U = _f32(U)
    al = np.float32(1.0 / (np.sqrt(np.sum(U.astype(np.float64) ** 2)) + eps_ns))
    X0 = (rnd if rnd_x0 is None else rnd_x0)(U)

    def poly(A):
        return rnd(b * A + c * (A @ A))

    def congruence(A, B):      # (aI + B) A (aI + B) for commuting symmetric A, B
        Z = rnd(a * A + A @ B)
        return rnd(a * Z + Z @ B)

    A0 = rnd((X0 @ X0.T) * (al * al))
    B0 = poly(A0)
    A1 = congruence(A0, B0)
    B1 = poly(A1)
    Q = rnd(B1 @ B0 + a * B0 + a * B1)                  # P_1 P_0 - a^2 I
    A2 = congruence(A1, B1)
    B2 = poly(A2)
    Q = rnd(B2 @ Q + a * Q + (a * a) * B2)              # P_2 P_1 P_0 - a^3 I
    X3 = rnd(al * ((a * a * a) * X0 + Q @ X0))
    A3 = rnd(X3 @ X3.T)
    B3 = poly(A3)
    X4 = rnd(a * X3 + B3 @ X3)
    A4 = congruence(A3, B3) if last_gram_from_previous else rnd(X4 @ X4.T)
    B4 = poly(A4)
    return a * X4 + B4 @ X4


def rel_fro(got, ref):
    got = np.asarray(got, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))


def emulated_error(U, schedule, split_input=False):
    """Relative Frobenius error of the emulated bf16 NS5 of the oriented matrix
    U against the fp64 recurrence.  schedule: "printed", "gram" (iterations 1-3
    in Gram space) or "gram+rec" (also the last Gram matrix by recurrence).
    split_input: X_0 as the sum of two bf16 numbers (Gram-space orders only)."""
    ref = ns5_fp64(U)
    if schedule == "fp32":
        got = ns5_bf16_printed(U, rnd=_f32)
    elif schedule == "printed":
        assert not split_input
        got = ns5_bf16_printed(U)
    else:
        got = ns5_bf16_gramspace(U, schedule == "gram+rec", rnd_x0=bf16_split_round if split_input else None)
    return rel_fro(got, ref)


def library_schedule(shape, split_input=False):
    """The order of evaluation the library's default options pick for a stored
    shape (documented in include/prm.h under PRM_OPT_NS_GRAM_SPAN): padded to
    multiples of 256, Gram space from 1024 oriented rows and c >= 1.5 r on, the
    last Gram matrix by recurrence where also c > 2r.  With PRM_OPT_NS_SPLIT_INPUT
    every shape from 1024 padded rows on takes the Gram-space order, the smaller
    ones run in fp32."""
    r, c = min(shape), max(shape)
    rp, cp = -(-r // 256) * 256, -(-c // 256) * 256
    if split_input and rp < 1024:
        return "fp32"
    if rp >= 1024 and (split_input or 2 * cp >= 3 * rp):
        return "gram+rec" if cp > 2 * rp else "gram"
    return "printed"
