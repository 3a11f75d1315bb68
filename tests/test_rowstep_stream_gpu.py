"""GPU parity of the single-pass (streaming) row step of tall matrices against
the fp64 oracle, element by element, through the C ABI.  PRM_OPT_TALL_KERNEL = 2
forces the streaming kernel on every shape it can take, however small, so that
ragged slabs (rows not a multiple of the CTA count), ragged column panels
(cols not a multiple of 64), CTAs without rows and several matrices per group
are all covered; the launch count tells which kernel ran."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from tests import util as U

pytestmark = pytest.mark.gpu

# rows/148 CTAs: 1000 -> slabs of 7 rows (the last CTAs idle), 20000 -> 136, 4096 -> 28; 264 = 4 panels + 8 columns
TALL = [(1000, 264), (2048, 512), (129, 8), (40, 24), (300, 256), (4096, 1024), (20000, 72), (9000, 64), (25000, 8)]


def _check(shapes, nesterov, seed, tall_kernel=2, heavy=False, eps_row=1e-8, expect_launches=None):
    cfg = U.oracle_cfg(K=4, beta=0.95, nesterov=nesterov, lr=5e-3, wd=0.01, gamma=0.15, eps_row=eps_row)
    W, G, M = U.make_inputs(shapes, seed, "bf16", heavy=heavy)
    n = []
    Wg, Mg = U.gpu_step(shapes, W, G, M, t=1, cfg=cfg, io="bf16", check_mode=False, tall_kernel=tall_kernel, launches=n)
    if expect_launches is not None:
        assert n[0] == expect_launches, n
    for i in range(len(shapes)):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 1, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {shapes[i]}")
        U.assert_elementwise(Wg[i], Wr, True, f"param {shapes[i]}")
    return Wg, Mg


@pytest.mark.parametrize("shape", TALL)
def test_stream_single(shape):
    _check([shape], True, seed=sum(shape) % 1000, expect_launches=1)      # one launch, not three


def test_stream_groups_no_nesterov_and_wide_neighbours():
    shapes = [(2048, 512), (64, 256), (2048, 512), (1000, 264), (2048, 512), (1000, 264)]
    _check(shapes, False, seed=5, expect_launches=3)      # two tall groups, one wide group: one launch each


def test_stream_heavy_tailed_rows_and_clamp():
    _check([(4096, 512)], True, seed=6, heavy=True)
    # zero and tiny columns: only the decay acts / divided by eps
    shapes = [(2000, 16)]
    cfg = U.oracle_cfg(K=4, nesterov=True, lr=5e-3, wd=0.01, eps_row=1e-3)
    W, G, M = U.make_inputs(shapes, 7, "bf16")
    G[0][:, 3] = 0
    M[0][:, 3] = 0
    G[0][:, 5] = 1e-7
    M[0][:, 5] = 0
    Wg, Mg = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, tall_kernel=2)
    Wr, Mr = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    U.assert_elementwise(Wg[0], Wr, True, "param")
    U.assert_elementwise(Mg[0], Mr, False, "momentum")


def test_stream_is_bit_reproducible_and_agrees_with_two_passes():
    shapes = [(4096, 1024), (1000, 264)]
    cfg = U.oracle_cfg(K=4, nesterov=True)
    W, G, M = U.make_inputs(shapes, 8, "bf16")
    a = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, tall_kernel=2)
    b = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, tall_kernel=2)
    n = []
    c = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, tall_kernel=1, launches=n)
    assert n[0] == 6                                     # two passes and the column norms per group
    for x, y in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(x, y)
    for i in range(2):
        assert np.array_equal(a[1][i], c[1][i])          # the momentum does not depend on the kernel
        # both are bf16 roundings of nearly the same fp32 value: at most one bf16 ulp apart
        assert (np.abs(a[0][i] - c[0][i]) <= 2 * U.bf16_half_ulp(c[0][i]) * (1 + 1e-3) + 1e-5 * np.abs(c[0][i])).all()
        assert (a[0][i] != c[0][i]).mean() < 0.02


def test_stream_falls_back_where_a_slab_does_not_fit():
    # 40000 rows over 148 CTAs: slabs of 271 rows, more than one TMA box holds; fp32 storage; odd columns
    n = []
    cfg = U.oracle_cfg(K=4, nesterov=True)
    for shape, io in (((40000, 8), "bf16"), ((2048, 512), "fp32"), ((300, 12), "bf16")):
        W, G, M = U.make_inputs([shape], 9, io)
        Wg, Mg = U.gpu_step([shape], W, G, M, 1, cfg, io, False, tall_kernel=2, launches=n)
        Wr, Mr = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
        U.assert_elementwise(Wg[0], Wr, io == "bf16", f"param {shape}")
    assert n == [3, 3, 3]


def test_stream_many_steps_on_one_handle_and_moved_buffers():
    """Several row steps on one handle (the per-wave counters are reset by every launch), then
    the same handle on other buffers (the tensor maps are rewritten)."""
    shape = (3000, 520)
    cfg = U.oracle_cfg(K=100, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs([shape], 10, "bf16")
    opt = B.PeriodicRowwiseMuon([shape], cfg.K, cfg.beta, cfg.nesterov, cfg.lr, cfg.wd, tall_kernel=2)
    for trial in range(2):
        w, g, m = U.Guarded(W[0]), U.Guarded(G[0]), U.Guarded(M[0])
        Wr, Mr = U.to_np64(W[0]), U.to_np64(M[0])
        for t in range(1, 5):
            opt.step([w.t], [g.t], [m.t], t)
            Wr, Mr = O.step_matrix(Wr, U.to_np64(G[0]), Mr, t, cfg)
        torch.cuda.synchronize()
        assert opt.status() == B.PRM_OK
        assert w.intact() and g.intact() and m.intact()
        U.assert_elementwise(U.to_np64(m.t), Mr, False, "momentum after four steps", rtol=4e-5)
        # four bf16 stores in a row: compare with four half-ulps
        assert np.abs(U.to_np64(w.t) - Wr).max() <= 4 * U.bf16_half_ulp(Wr).max() + 1e-6
    opt.close()
