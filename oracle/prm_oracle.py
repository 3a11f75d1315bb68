"""fp64 CPU oracle for the Periodic Row-wise Muon optimizer step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the
CUDA library is compared against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does, and
this module imports nothing from the CUDA package.  It shares no code, table
or constant generator with the kernels.

Everything is float64 numpy.  Each function follows one passage of the paper
("Scaling Muon for Diffusion Transformers"), named in its docstring.  The
steps are written in the paper's order and notation; the only library
primitive used as a step is numpy's matrix product.

Readings of the paper taken here (the paper is silent or ambiguous on them):

* Momentum recurrence (Algorithm 1 line 2 points at Section 2, which gives no
  formula): exponential moving average  M_t = beta*M_{t-1} + (1-beta)*G_t,
  M_{-1} = 0.  The update direction is invariant to the EMA-vs-accumulate
  choice (both branches remove global scale); only the stored buffer differs
  by the constant (1-beta).  Buffer convention: parity unpinned.
* Nesterov: not in the paper (it uses "the current momentum M_t").  With
  nesterov=False the direction input is U = M_t (paper-literal); with
  nesterov=True it is U = beta*M_t + (1-beta)*G_t.  Parity unpinned.
* NS5 input normalisation (the paper only names "the input normalization"):
  X_0 = X / (||X||_F + eps_ns).  Value of eps_ns: parity unpinned.
* Shape scale s(W) (named, never defined): a function of the stored shape
  (m, n) only; see shape_scale().  Parity unpinned.
* RowNorm epsilon: form max(||row||, eps) with the square root taken before
  the clamp is the paper's; the value 1e-8 is a choice.  Parity unpinned.

Functions with a pin (tests/test_oracle_pins.py): momentum_update,
direction_input, orient, orient_inv, rownorm, ns5, is_refresh,
group_by_shape, step_matrix (decay term, learning-rate scaling, branch
selection, gamma placement), shard_rows (torch.chunk), pipeline_time (event
simulation), refresh_from_shards (equals the dense step), bucket_plan (plan
invariants only: the paper gives no bucketing rule, parity unpinned).
"""

from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

# Newton-Schulz coefficients and iteration count (Appendix "Optimizer and
# Training Hyperparameters": five iterations, (a, b, c) fixed).
NS_A = 3.4445
NS_B = -4.7750
NS_C = 2.0315
NS_ITERS = 5


@dataclass
class OracleConfig:
    """Hyper-parameters of Algorithm 1's matrix branch."""

    K: int = 3                # refresh period (Section 3.2), K >= 1
    beta: float = 0.95        # momentum coefficient (hyper-parameter table)
    nesterov: bool = False
    lr: float = 5e-3          # eta_t
    wd: float = 0.01          # lambda, decoupled weight decay
    gamma: float = 0.15       # RowNorm multiplier (Section 3.2)
    eps_row: float = 1e-8     # epsilon of Eq. (rownorm)
    eps_ns: float = 1e-7      # epsilon of the NS5 input normalisation
    scale_mode: int = 1       # see shape_scale()
    # Ablation variants of the paper's Table 3(a):
    gamma_ns: float = 1.0     # multiplier on the NS5 branch ("scalar-controlled" sets it to gamma)
    no_refresh: bool = False  # RowNorm at every step (no NS5 schedule)


def is_refresh(t: int, K: int) -> bool:
    """Refresh indicator rho_t = 1[t mod K == 0], t zero-based (Section 3.2;
    Algorithm 1 line 3)."""
    if K < 1:
        raise ValueError("K must be >= 1")
    return (t % K) == 0


def group_by_shape(shapes):
    """Group matrices by exact stored shape (rows, cols).

    Returns (group_of_mat, order_in_group, group_shapes).  Group ids follow
    first appearance in the caller's list; inside a group the caller's order
    is kept.  (a, b) and (b, a) are different groups.
    """
    group_shapes = []
    group_of_mat = []
    order_in_group = []
    counts = []
    for (m, n) in shapes:
        key = (int(m), int(n))
        if key not in group_shapes:
            group_shapes.append(key)
            counts.append(0)
        g = group_shapes.index(key)
        group_of_mat.append(g)
        order_in_group.append(counts[g])
        counts[g] += 1
    return group_of_mat, order_in_group, group_shapes


def momentum_update(M_prev, G, beta):
    """M_t = beta*M_{t-1} + (1-beta)*G_t (Algorithm 1 line 2, EMA reading)."""
    M_prev = np.asarray(M_prev, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    return beta * M_prev + (1.0 - beta) * G


def direction_input(M_t, G, beta, nesterov):
    """Matrix handed to the direction map: the current momentum M_t
    (Section 3.2, "at every step we use the current momentum"), or its
    Nesterov look-ahead beta*M_t + (1-beta)*G_t when nesterov is set."""
    M_t = np.asarray(M_t, dtype=np.float64)
    if not nesterov:
        return M_t.copy()
    return beta * M_t + (1.0 - beta) * np.asarray(G, dtype=np.float64)


def orient(U):
    """Orientation map O: U itself if m <= n, else its transpose, so that the
    result is r x c with r = min(m, n) <= c (Section 3.1)."""
    m, n = U.shape
    return U if m <= n else U.T


def orient_inv(D_tilde, m, n):
    """Inverse orientation: map an r x c direction back to the stored m x n
    shape (Section 3.1)."""
    return D_tilde if m <= n else D_tilde.T


def rownorm(X, eps):
    """RowNorm_eps(X)_i = X_i / max(||X_i||_2, eps)  (Eq. rownorm; Appendix
    Eq. app-rownorm-eps).  Square root first, then the clamp (Algorithm 2
    line 12)."""
    X = np.asarray(X, dtype=np.float64)
    out = np.empty_like(X)
    for i in range(X.shape[0]):
        row = X[i]
        q = float(np.sum(row * row))
        nu = max(math.sqrt(q), eps)
        out[i] = row / nu
    return out


def ns5(X, eps_ns, iters=NS_ITERS):
    """Finite Newton-Schulz map Phi_5 on an oriented r x c matrix (r <= c):
    X_0 = X/(||X||_F + eps_ns), then for j = 0..4
        G_j = X_j X_j^T,  B_j = b*G_j + c*G_j^2,  X_{j+1} = a*X_j + B_j X_j
    (Appendix Eq. app-ns-recurrence with the fixed coefficients).  This is
    the iteration itself, not the polar factor."""
    X = np.asarray(X, dtype=np.float64)
    fro = math.sqrt(float(np.sum(X * X)))
    Xj = X / (fro + eps_ns)
    for _ in range(iters):
        Gj = Xj @ Xj.T
        Bj = NS_B * Gj + NS_C * (Gj @ Gj)
        Xj = NS_A * Xj + Bj @ Xj
    return Xj


def shape_scale(m, n, mode):
    """Shape-dependent update scale s(W) of Eq. (finite_ns5).  The paper
    never defines it; it depends on the stored shape only.
      mode 0: 1
      mode 1: sqrt(max(1, m/n))
      mode 2: 0.2*sqrt(max(m, n))
    """
    if mode == 0:
        return 1.0
    if mode == 1:
        return math.sqrt(max(1.0, float(m) / float(n)))
    if mode == 2:
        return 0.2 * math.sqrt(float(max(m, n)))
    raise ValueError("unknown scale mode")


def direction(U, refresh, cfg: OracleConfig):
    """D_tilde of Eq. (periodic-direction) mapped back to the stored shape:
    NS5(O(U)) on a refresh step, gamma*RowNorm_eps(O(U)) otherwise."""
    m, n = U.shape
    U_tilde = orient(U)
    if refresh:
        D_tilde = cfg.gamma_ns * ns5(U_tilde, cfg.eps_ns)
    else:
        D_tilde = cfg.gamma * rownorm(U_tilde, cfg.eps_row)
    return orient_inv(D_tilde, m, n)


def step_matrix(W, G, M_prev, t, cfg: OracleConfig):
    """One step of Algorithm 1 for one matrix of the Muon set.

    W, G, M_prev: stored m x n arrays (any float dtype; widened to fp64).
    Returns (W_next, M_t) in fp64.
    """
    W = np.asarray(W, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    m, n = W.shape
    M_t = momentum_update(M_prev, G, cfg.beta)                 # line 2
    U = direction_input(M_t, G, cfg.beta, cfg.nesterov)
    refresh = is_refresh(t, cfg.K) and not cfg.no_refresh       # line 3
    D = shape_scale(m, n, cfg.scale_mode) * direction(U, refresh, cfg)  # lines 5-8
    W_next = (1.0 - cfg.lr * cfg.wd) * W - cfg.lr * D           # line 9
    return W_next, M_t


def step(params, grads, momenta, t, cfg: OracleConfig):
    """Algorithm 1 lines 4-10 over a list of matrices.  Returns two lists."""
    W_out, M_out = [], []
    for W, G, M in zip(params, grads, momenta):
        Wn, Mn = step_matrix(W, G, M, t, cfg)
        W_out.append(Wn)
        M_out.append(Mn)
    return W_out, M_out


def adamw_step(p, g, m, v, t, lr=1e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.01):
    """One AdamW step for a parameter outside the Muon set (Algorithm 1 line 11
    leaves those to the baseline's AdamW; hyper-parameter table: lr 1e-4,
    betas (0.9, 0.95), eps 1e-8, weight decay 0.01).  The paper does not spell
    the rule out; this is the usual decoupled form with bias correction:
        p <- p*(1 - lr*wd)
        m <- beta1*m + (1-beta1)*g,   v <- beta2*v + (1-beta2)*g^2
        p <- p - lr * (m/(1-beta1^t)) / (sqrt(v/(1-beta2^t)) + eps)
    with t the 1-based step count.  Returns (p, m, v) in fp64."""
    p = np.asarray(p, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    p = p * (1.0 - lr * wd)
    m_hat = m / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    p = p - lr * m_hat / (np.sqrt(v_hat) + eps)
    return p, m, v


# --------------------------------------------------------------------------
# Distributed execution of the refresh branch (Section 3.3; Algorithm 2 lines
# 1-7; appendix "Idealized overlap model").  Host-side planning and the
# reference result of a refresh computed from row shards.
#
# Readings taken here (the paper only says that the Muon matrices are
# partitioned into communication buckets and that FSDP2 shards dim 0):
# * rows are split as torch.chunk splits them, chunk = ceil(rows / world);
# * buckets are filled greedily, walking the matrices shape group by shape
#   group (so that a bucket holds same-shape matrices, which NS5 batches); a
#   matrix is never split, and a bucket is closed when the gathered payload
#   (world segments of 2-byte elements) would exceed the byte cap; every
#   matrix's slot in a segment is rounded up to 8 elements.  Parity unpinned against the paper
#   (it gives no rule); pinned by the invariants every valid plan must have.


def shard_rows(rows, world, rank):
    """(start, count) of rank's rows under dim-0 sharding (Section 3.3)."""
    chunk = -(-rows // world)
    lo = min(rows, rank * chunk)
    hi = min(rows, lo + chunk)
    return lo, hi - lo


def bucket_plan(shapes, world, bucket_bytes):
    """Communication buckets B_l of Algorithm 2: (bucket_of_mat, offset_in_segment, segment_elems).
    The matrices are walked shape group by shape group (groups in order of first
    appearance, given order inside a group)."""
    groups = group_by_shape(shapes)[0]
    walk = sorted(range(len(shapes)), key=lambda i: (groups[i], i))
    bucket_of_mat, offsets, segments = [None] * len(shapes), [None] * len(shapes), []
    seg = 0
    for i in walk:
        m, n = shapes[i]
        chunk = -(-m // world)
        need = -(-(chunk * n) // 8) * 8
        if seg > 0 and (seg + need) * 2 * world > bucket_bytes:
            segments.append(seg)
            seg = 0
        bucket_of_mat[i] = len(segments)
        offsets[i] = seg
        seg += need
    segments.append(seg)
    return bucket_of_mat, offsets, segments


def pipeline_time(a, c):
    """(T_pipe, T_comm_exposed) of the ideal two-stage pipeline over buckets with
    all-gather times a_l and compute times c_l (Eq. app-pipeline-time and
    Eq. app-exposed-communication)."""
    B = len(a)
    t_pipe = a[0] + sum(max(c[l], a[l + 1]) for l in range(B - 1)) + c[B - 1]
    t_exposed = a[0] + sum(max(0.0, a[l + 1] - c[l]) for l in range(B - 1))
    return t_pipe, t_exposed


def refresh_from_shards(W_shards, G_shards, M_shards, cfg: OracleConfig):
    """Algorithm 2 lines 1-7 for one matrix, all ranks at once: every rank
    updates the momentum of its rows, the rows are gathered into the full
    momentum (here: concatenated), NS5 runs on the full matrix, and each rank
    keeps its rows of the result.  Returns (new W shards, new M shards)."""
    M_new = [momentum_update(M, G, cfg.beta) for M, G in zip(M_shards, G_shards)]
    U_full = np.concatenate([direction_input(M, G, cfg.beta, cfg.nesterov) for M, G in zip(M_new, G_shards)], axis=0)
    m, n = U_full.shape
    D = shape_scale(m, n, cfg.scale_mode) * direction(U_full, True, cfg)
    out, lo = [], 0
    for W in W_shards:
        hi = lo + W.shape[0]
        out.append((1.0 - cfg.lr * cfg.wd) * W - cfg.lr * D[lo:hi])
        lo = hi
    return out, M_new
