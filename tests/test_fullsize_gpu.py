"""Parity at the benchmark's full sizes, in the launch configuration that
bench.py times (one handle over the whole shape set, default options).

The oracle cannot run every matrix of these shape sets, so each case checks
  * the row step on sampled stored rows (wide) and stored columns (tall) of
    sampled matrices against the oracle, element by element;
  * the refresh on one whole block (one matrix of every shape): tensor-core
    result against the fp32 check mode and against the fp64 oracle, for all
    five shapes of every configuration;
  * the refresh on every matrix of the set: the Frobenius norm of the
    direction, which NS5 leaves near sqrt(r);
  * the row step on every matrix of the set: the norm of every oriented row
    of the update, which RowNorm fixes at lr*s*gamma.
Configuration 5 keeps 168.8 GiB resident at its stated 48 blocks.  The test
asks the device how much memory is free and runs the largest block count that
fits (workloads.blocks_that_fit, the same call bench.py makes), with the NS5
workspace capped at 2 GiB; on a B200 with ~177.7 GiB free that is all 48.
Everything the test itself needs beside the shape set (copies of the sampled
matrices, the check-mode workspace) is kept on the host or sized for one
matrix at a time.
"""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from paper_2608_20818_b200.workloads import (NS_WORKSPACE_BYTES_WHEN_FULL, blocks_that_fit, make_grad, make_momentum,
                                             make_param, workload)
from tests import util as U

pytestmark = pytest.mark.gpu


def _oracle_cfg(wl):
    return O.OracleConfig(K=wl.K, beta=wl.beta, nesterov=wl.nesterov, lr=wl.lr, wd=wl.wd, gamma=wl.gamma)


def _check_row_step_samples(wl, idx, W0, M0, G, W1, M1, rng):
    """Sampled rows (wide) or columns (tall) of matrix idx against the oracle."""
    cfg = _oracle_cfg(wl)
    m, n = wl.shapes[idx]
    s = O.shape_scale(m, n, cfg.scale_mode)
    decay = 1.0 - cfg.lr * cfg.wd
    if m <= n:
        rows = rng.choice(m, size=8, replace=False)
        for r in rows:
            w0, m0, g = (U.to_np64(x[r:r + 1]) for x in (W0, M0, G))
            mt = O.momentum_update(m0, g, cfg.beta)
            u = O.direction_input(mt, g, cfg.beta, cfg.nesterov)
            want = decay * w0 - cfg.lr * s * cfg.gamma * O.rownorm(u, cfg.eps_row)
            U.assert_elementwise(U.to_np64(M1[r:r + 1]), mt, False, f"momentum row {r} of {idx}")
            U.assert_elementwise(U.to_np64(W1[r:r + 1]), want, True, f"param row {r} of {idx}")
    else:
        cols = rng.choice(n, size=8, replace=False)
        for c in cols:
            w0, m0, g = (U.to_np64(x[:, c:c + 1]).T for x in (W0, M0, G))     # 1 x m oriented rows
            mt = O.momentum_update(m0, g, cfg.beta)
            u = O.direction_input(mt, g, cfg.beta, cfg.nesterov)
            want = decay * w0 - cfg.lr * s * cfg.gamma * O.rownorm(u, cfg.eps_row)
            U.assert_elementwise(U.to_np64(M1[:, c:c + 1]).T, mt, False, f"momentum col {c} of {idx}")
            U.assert_elementwise(U.to_np64(W1[:, c:c + 1]).T, want, True, f"param col {c} of {idx}")


def _run_config(config_id, blocks, oracle_shapes, ns_workspace_bytes=None):
    wl = workload(config_id, blocks)
    n = len(wl.shapes)
    dev = "cuda"
    rng = np.random.default_rng(config_id)
    params = [make_param(wl, i, dev) for i in range(n)]
    moms = [make_momentum(wl, i, dev) for i in range(n)]
    grads = [make_grad(wl, i, 0, dev) for i in range(n)]
    opt = B.PeriodicRowwiseMuon(wl.shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma,
                                ns_workspace_bytes=ns_workspace_bytes)
    block = int(rng.integers(0, n // 5))
    sample = list(range(5 * block, 5 * block + 5))            # one matrix of every shape

    # ---- row step (t = 1), from momentum made non-zero by a first row step (t = 2 of another period)
    opt.step(params, grads, moms, 2)
    pre = {i: (params[i].cpu(), moms[i].cpu()) for i in sample}   # host copies: the device may be full
    opt.step(params, grads, moms, 1)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for i in sample:
        _check_row_step_samples(wl, i, pre[i][0], pre[i][1], grads[i].cpu(), params[i].cpu(), moms[i].cpu(), rng)
    del pre

    # ---- refresh (t = K).  All parameters start from zero, so the step writes -lr*s*NS5(U) and
    # the bf16 store keeps 2^-9 relative precision on the direction itself.
    for p in params:
        p.zero_()
    pre = {i: moms[i].cpu() for i in sample}
    opt.step(params, grads, moms, wl.K)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    # Every matrix of the set, whatever sub-batch it was refreshed in: five NS5 iterations leave the
    # singular values of a well-spread spectrum in a band around one, so ||NS5(U)||_F / sqrt(r) is
    # of order one (heavy-tailed inputs keep a few small singular values: lower edge 0.3).
    for i, (m, k) in enumerate(wl.shapes):
        sc = O.shape_scale(m, k, 1)
        ratio = float(torch.linalg.norm(params[i].float())) / (wl.lr * sc * min(m, k) ** 0.5)
        assert 0.3 <= ratio <= 1.2, (i, (m, k), ratio)
    # the same five matrices through the fp32 check mode, one at a time (its fp32 workspace is
    # twice the size of the tensor-core path's) and through the fp64 oracle
    cfg = _oracle_cfg(wl)
    out = {}
    for i in sample:
        shape = wl.shapes[i]
        torch.cuda.empty_cache()               # temporaries of the norm loop above: the device may be nearly full
        chk = B.PeriodicRowwiseMuon([shape], wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma, check_mode=True)
        Wc = torch.zeros_like(params[i])
        Mc = pre[i].to(dev)
        chk.step([Wc], [grads[i]], [Mc], wl.K)
        torch.cuda.synchronize()
        assert chk.status() == B.PRM_OK
        chk.close()
        del chk
        assert torch.equal(Mc, moms[i]), "momentum must not depend on the NS5 mode"
        del Mc
        W_fast, W_chk = U.to_np64(params[i]), U.to_np64(Wc)
        del Wc
        torch.cuda.empty_cache()
        assert np.abs(W_chk).max() > 0
        err = U.rel_fro(W_fast, W_chk)
        out[shape] = err
        assert err <= 2e-2, (shape, err)
        if shape in oracle_shapes:
            Wr, Mr = O.step_matrix(np.zeros(shape), U.to_np64(grads[i]), U.to_np64(pre[i]), wl.K, cfg)
            U.assert_elementwise(U.to_np64(moms[i]), Mr, False, f"momentum {shape}")
            e_fast = U.rel_fro(W_fast, Wr)
            e_chk = U.rel_fro(W_chk, Wr)
            print(f"config {config_id} {shape}: tensor-core path {e_fast:.3e}, check mode {e_chk:.3e} against the oracle")
            assert e_fast <= 2e-2, (shape, e_fast)
            assert e_chk <= 4e-3, (shape, e_chk)       # fp32 arithmetic, bf16 store (2^-9)
    del pre
    # ---- row step from zero parameters on every matrix of the set: the step writes
    # -lr*s*gamma*RowNorm(U), so every oriented row (stored row of a wide matrix, stored column of a
    # tall one) has norm lr*s*gamma, up to the bf16 rounding of its entries.
    for p in params:
        p.zero_()
    opt.step(params, grads, moms, 1)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for i, (m, k) in enumerate(wl.shapes):
        want = wl.lr * O.shape_scale(m, k, 1) * wl.gamma
        norms = torch.linalg.vector_norm(params[i].float(), dim=1 if m <= k else 0)
        assert float((norms / want - 1).abs().max()) <= 2e-3, (i, (m, k))
    opt.close()
    return out


def _all_shapes(d):
    return {(d, 3 * d), (d, d), (d, 4 * d), (4 * d, d), (d, 6 * d)}


def test_config2_full():
    _run_config(2, None, _all_shapes(2048))


def test_config3_full():
    _run_config(3, None, _all_shapes(3072))


def test_config4_full():
    _run_config(4, None, _all_shapes(4096))


def test_config5_heavy_tailed_rows_largest_block_count_that_fits():
    import gc
    gc.collect()
    torch.cuda.empty_cache()                  # what earlier tests left in torch's cache counts as free
    free, total = torch.cuda.mem_get_info()
    blocks = blocks_that_fit(5, free)
    print(f"configuration 5: {free / 2**30:.2f} GiB free of {total / 2**30:.2f} GiB -> {blocks} of 48 blocks "
          f"({blocks * 18 * 5120**2 * 8 / 2**30:.2f} GiB resident)")
    assert blocks >= 40, "a B200 with its memory free holds at least 40 of the 48 blocks"
    _run_config(5, blocks, _all_shapes(5120), ns_workspace_bytes=NS_WORKSPACE_BYTES_WHEN_FULL)


def test_check_mode_direction_at_4096():
    """fp32 check mode against the oracle at d = 4096 with fp32 parameters
    (W = 0, lr = 1: the step writes the direction itself)."""
    shapes = [(4096, 4096)]
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=1.0, wd=0.0, scale_mode=0)
    W, G, M = U.make_inputs(shapes, 4096, "fp32", grad_std=1e-3, mom_std=1e-3)
    W[0].zero_()
    for mode, tol in ((True, 1e-4), (False, 2e-2)):
        Wg, _ = U.gpu_step(shapes, W, G, M, 0, cfg, "fp32", mode)
        Wr, _ = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 0, cfg)
        err = U.rel_fro(Wg[0], Wr)
        assert err <= tol, (mode, err)


def test_split_input_on_one_block_of_the_9b_class_set():
    """PRM_OPT_NS_SPLIT_INPUT at the benchmark's matrix sizes: one matrix of every d = 4096 shape,
    the two-plane tensor-core refresh against the fp32 check mode, and against the fp64 oracle on
    the square matrix (the one shape whose order of evaluation the option changes)."""
    d = 4096
    shapes = [(d, 3 * d), (d, d), (d, 4 * d), (4 * d, d), (d, 6 * d)]
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=1.0, wd=0.0, scale_mode=0)
    W, G, M = U.make_inputs(shapes, 4097, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    Ws, Ms = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", False, split_input=True)
    Wc, Mc = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", True)
    for i, s in enumerate(shapes):
        assert np.array_equal(Ms[i], Mc[i]), s
        err = U.rel_fro(Ws[i], Wc[i])
        assert err <= 2e-2, (s, err)
    Wr, _ = O.step_matrix(U.to_np64(W[1]), U.to_np64(G[1]), U.to_np64(M[1]), 0, cfg)
    err = U.rel_fro(Ws[1], Wr)
    assert err <= 2e-2, err
