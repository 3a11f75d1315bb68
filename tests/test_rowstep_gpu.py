"""GPU parity: the row-wise branch (rho_t = 0) against the fp64 oracle,
element by element, through the C ABI."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from tests import util as U

pytestmark = pytest.mark.gpu

# Each shape exercises one launch variant.  bf16 rows of up to 24576 elements with cols % 8 == 0
# take the persistent kernel (1 to 6 chunks of 4096 elements, the last one ragged; more rows than
# CTAs; fewer rows than CTAs); fp32 storage, longer rows and PRM_OPT_WIDE_KERNEL = 1 take one CTA
# per row with 1 to 4 vectors per thread, clusters beyond 32768 elements, the generic kernel for
# unaligned or still longer rows; tall matrices with ragged row blocks.
WIDE = [(256, 1024), (8, 16), (24, 40), (10, 36), (5, 5), (1, 8), (300, 2056), (33, 4104), (20, 8200),
        (12, 16392), (6, 32776), (3, 70000), (2, 65536), (7, 30720), (7, 24576), (3, 24568), (500, 4096),
        (5, 12288)]
TALL = [(40, 24), (36, 10), (1000, 264), (2048, 512), (129, 8), (300, 257), (16, 1)]


def _check(shapes, io, nesterov, seed, heavy=False, eps_row=1e-8, mom_std=0.1, grad_std=1.0, wide_kernel=0):
    cfg = U.oracle_cfg(K=4, beta=0.95, nesterov=nesterov, lr=5e-3, wd=0.01, gamma=0.15, eps_row=eps_row)
    W, G, M = U.make_inputs(shapes, seed, io, heavy=heavy, mom_std=mom_std, grad_std=grad_std)
    Wg, Mg = U.gpu_step(shapes, W, G, M, t=1, cfg=cfg, io=io, check_mode=True, wide_kernel=wide_kernel)
    for i in range(len(shapes)):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 1, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {shapes[i]}")
        U.assert_elementwise(Wg[i], Wr, io == "bf16", f"param {shapes[i]}")


@pytest.mark.parametrize("shape", WIDE + TALL)
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_rowstep_single(shape, io):
    _check([shape], io, nesterov=True, seed=hash(shape) % 1000)


@pytest.mark.parametrize("shape", [s for s in WIDE if s[1] % 8 == 0 and s[1] <= 24576])
def test_rowstep_wide_one_row_per_cta(shape):
    """PRM_OPT_WIDE_KERNEL = 1: the bf16 shapes that the persistent kernel takes by default."""
    _check([shape], "bf16", nesterov=True, seed=hash(shape) % 1000, wide_kernel=1)


def test_rowstep_wide_kernels_agree_and_groups_share_a_launch():
    """Three groups with several matrices each (more rows than CTAs, rows round robin over the
    CTAs across matrix boundaries): both wide kernels against the oracle, the same momentum bit
    for bit, parameters within one bf16 rounding of each other."""
    shapes = [(300, 2056), (64, 256), (300, 2056), (40, 8200), (300, 2056), (64, 256), (40, 8200)]
    cfg = U.oracle_cfg(K=4, nesterov=False, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 15, "bf16")
    res = []
    for wk in (0, 1):
        n = []
        Wg, Mg = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", True, wide_kernel=wk, launches=n)
        assert n[0] == 3, n
        for i in range(len(shapes)):
            Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 1, cfg)
            U.assert_elementwise(Mg[i], Mr, False, f"momentum {shapes[i]}")
            U.assert_elementwise(Wg[i], Wr, True, f"param {shapes[i]}")
        res.append((Wg, Mg))
    for i in range(len(shapes)):
        assert np.array_equal(res[0][1][i], res[1][1][i])
        a, b = res[0][0][i], res[1][0][i]
        assert (np.abs(a - b) <= 2 * U.bf16_half_ulp(b) * (1 + 1e-3) + 1e-5 * np.abs(b)).all()


@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_rowstep_no_nesterov_mixed_groups(io):
    shapes = [(64, 256), (256, 64), (64, 256), (48, 48), (256, 64), (64, 256), (10, 36)]
    _check(shapes, io, nesterov=False, seed=5)


def test_rowstep_heavy_tailed_rows():
    _check([(512, 2048), (2048, 512)], "bf16", nesterov=True, seed=6, heavy=True, grad_std=1e-3, mom_std=1e-3)


def test_rowstep_zero_and_tiny_rows():
    # zero direction input: only the decay acts; tiny rows are divided by eps
    shapes = [(4, 16), (16, 4)]
    cfg = U.oracle_cfg(K=4, nesterov=True, lr=5e-3, wd=0.01, eps_row=1e-3)
    W, G, M = U.make_inputs(shapes, 7, "fp32")
    for i in range(2):
        G[i].zero_()
        M[i].zero_()
    G[0][1] = 1e-6   # row norm 4e-6*... < eps
    G[1][:, 2] = 1e-6
    Wg, Mg = U.gpu_step(shapes, W, G, M, 1, cfg, "fp32", True)
    for i in range(2):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 1, cfg)
        U.assert_elementwise(Wg[i], Wr, False, "param")
        U.assert_elementwise(Mg[i], Mr, False, "momentum")
    np.testing.assert_allclose(Wg[0][0], (1 - 5e-3 * 0.01) * U.to_np64(W[0])[0], rtol=1e-6)


@pytest.mark.parametrize("wide_kernel", [0, 1])
def test_rowstep_zero_and_tiny_rows_bf16(wide_kernel):
    """The same degenerate rows through the bf16 kernels (persistent and one row per CTA): a zero
    row only decays, a tiny row is divided by eps_row, a row of one huge element keeps its sign."""
    shapes = [(6, 4104)]
    cfg = U.oracle_cfg(K=4, nesterov=True, lr=5e-3, wd=0.01, eps_row=1e-3)
    W, G, M = U.make_inputs(shapes, 17, "bf16")
    G[0][0].zero_(); M[0][0].zero_()
    G[0][1].zero_(); M[0][1].zero_(); G[0][1, 7] = 1e-6
    G[0][2].zero_(); M[0][2].zero_(); G[0][2, 4100] = -3e4
    Wg, Mg = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", True, wide_kernel=wide_kernel)
    Wr, Mr = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    U.assert_elementwise(Wg[0], Wr, True, "param")
    U.assert_elementwise(Mg[0], Mr, False, "momentum")


def test_rowstep_run_to_run_bit_identical():
    shapes = [(300, 2056), (1000, 264), (6, 32776)]
    cfg = U.oracle_cfg(K=4, nesterov=True)
    W, G, M = U.make_inputs(shapes, 8, "bf16")
    a = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", True)
    b = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", True)
    for x, y in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(x, y)


def test_misaligned_pointer_is_refused():
    from paper_2608_20818_b200 import binding as B
    opt = B.PeriodicRowwiseMuon([(8, 16)], 4, check_mode=True)
    buf = torch.zeros(8 * 16 + 8, dtype=torch.bfloat16, device="cuda")
    bad = buf[1:1 + 128].view(8, 16)
    good = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(8, 16, device="cuda")
    with pytest.raises(B.PrmError) as e:
        opt.step([bad], [good], [m], 1)
    assert e.value.code == B.PRM_ERR_ALIGN
    opt.close()
