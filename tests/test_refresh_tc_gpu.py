"""GPU parity of the tensor-core refresh (bf16 operands, fp32 accumulation in
tensor memory) against the fp64 oracle: relative Frobenius error of the NS5
direction at most 2e-2 per matrix."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from tests import util as U
from tests.test_refresh_check_gpu import _config1_trajectory, _direction_case

pytestmark = pytest.mark.gpu

TOL = 2e-2
SHAPES = [(256, 512), (256, 1024), (24, 40), (40, 24), (300, 520), (512, 256), (5, 5), (130, 1000),
          (768, 768), (1024, 3072), (2048, 512)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_refresh_tc_direction(shape, io):
    (err,) = _direction_case([shape], io, False, seed=sum(shape))
    # A 5x5 matrix has too few entries for bf16 rounding to average out: the
    # same arithmetic that gives ~1e-2 on real shapes scatters between 1e-2
    # and 3e-2 there, so the tiny case gets twice the bound.
    assert err <= (TOL if min(shape) >= 16 else 2 * TOL), err


def test_refresh_tc_groups_and_sub_batches():
    shapes = [(256, 512), (512, 256), (256, 512), (256, 256), (256, 512), (512, 256), (512, 768)]
    errs = _direction_case(shapes, "bf16", False, seed=3, ns_ws=1)
    assert max(errs) <= TOL, errs
    errs = _direction_case(shapes, "bf16", False, seed=3, nesterov=False)
    assert max(errs) <= TOL, errs


def _structured_case(kind, shapes, check_mode):
    g = torch.Generator().manual_seed(5)
    cfg = U.oracle_cfg(K=1, nesterov=True, lr=1.0, wd=0.0, scale_mode=0)
    W = [torch.zeros(s, dtype=torch.bfloat16) for s in shapes]
    G = []
    for (m, n) in shapes:
        if kind == "heavy_rows":          # log-normal row scales, as in the 15B-class configuration
            x = torch.randn(m, n, generator=g) * torch.exp(torch.randn(m, 1, generator=g))
        elif kind == "low_rank_mild":     # rank-8 signal at the level of the noise
            x = torch.randn(m, 8, generator=g) @ torch.randn(8, n, generator=g) / 8 ** 0.5 + torch.randn(m, n, generator=g)
        else:                             # rank-8 spike two orders of magnitude above the noise floor
            x = torch.randn(m, 8, generator=g) @ torch.randn(8, n, generator=g) + 0.1 * torch.randn(m, n, generator=g)
        G.append((x * 1e-3).to(torch.bfloat16))
    M = [torch.zeros(s) for s in shapes]
    Wg, _ = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", check_mode)
    errs = []
    for i in range(len(shapes)):
        Wr, _ = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        errs.append(U.rel_fro(Wg[i], Wr))
    return errs


@pytest.mark.parametrize("kind", ["heavy_rows", "low_rank_mild"])
def test_refresh_tc_structured_inputs(kind):
    errs = _structured_case(kind, [(512, 1024), (1024, 512)], False)
    assert max(errs) <= TOL, errs


def test_refresh_tc_spiked_spectrum_is_bf16_limited():
    # With a few singular values far above the rest, the bf16 rounding of the
    # dominant part is of the order of the small singular values, and NS5
    # amplifies those by ~3.4x per iteration.  That is a property of bf16
    # operands, not of the kernels: the result stays within 10 % here, and the
    # fp32 check mode (params stored as bf16 here) is two orders better.
    shapes = [(512, 1024)]
    fast = _structured_case("spiked", shapes, False)
    check = _structured_case("spiked", shapes, True)
    assert max(fast) <= 0.1, fast
    assert max(check) <= 3e-3, check


def test_refresh_tc_matches_check_mode_and_is_reproducible():
    shapes = [(512, 1536), (1536, 512), (512, 1536)]
    cfg = U.oracle_cfg(K=2, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 9, "fp32", grad_std=1e-3, mom_std=1e-3)
    a = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", False)
    b = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", False)
    c = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", True)
    for i in range(3):
        assert np.array_equal(a[0][i], b[0][i]) and np.array_equal(a[1][i], b[1][i])
        assert np.array_equal(a[1][i], c[1][i])            # momentum does not depend on the NS5 mode
        w0 = U.to_np64(W[i])
        d_fast = (1 - 5e-5) * w0 - a[0][i]
        d_chk = (1 - 5e-5) * w0 - c[0][i]
        assert U.rel_fro(d_fast, d_chk) <= TOL


def test_config1_eight_steps_tensor_cores():
    _config1_trajectory(False, TOL)


def test_refresh_tc_zero_matrix():
    shapes = [(64, 128)]
    cfg = U.oracle_cfg(K=1, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 12, "fp32")
    G[0].zero_()
    M[0].zero_()
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, "fp32", False)
    np.testing.assert_allclose(Wg[0], (1 - 5e-5) * U.to_np64(W[0]), rtol=1e-6)
