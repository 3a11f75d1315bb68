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
    assert err <= TOL, err
    if min(shape) < 64:
        # fewer than 64 oriented rows: the library refreshes in fp32 (bf16 scatters past
        # the bound there, tests/test_bf16_emulation.py), so the result is far inside it
        assert err <= (1e-4 if io == "fp32" else 3e-3), err      # bf16 parameters: the store rounds to 2^-9


def test_refresh_tc_groups_and_sub_batches():
    shapes = [(256, 512), (512, 256), (256, 512), (256, 256), (256, 512), (512, 256), (512, 768)]
    errs = _direction_case(shapes, "bf16", False, seed=3, ns_ws=1)
    assert max(errs) <= TOL, errs
    errs = _direction_case(shapes, "bf16", False, seed=3, nesterov=False)
    assert max(errs) <= TOL, errs


def _structured_case(kind, shapes, check_mode):
    cfg = U.oracle_cfg(K=1, nesterov=True, lr=1.0, wd=0.0, scale_mode=0)
    W = [torch.zeros(s, dtype=torch.bfloat16) for s in shapes]
    G = U.structured_grads(kind, shapes)
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


def spiked_bounds(shapes):
    """1.5 x the error that bf16 storage with fp32 accumulation gives on the
    very same bits, emulated on the CPU in the order of evaluation the library
    picks for each shape."""
    from tests import bf16_emulation as E
    from tests.test_bf16_emulation import direction_input_of
    return [1.5 * E.emulated_error(direction_input_of(g, s), E.library_schedule(s))
            for s, g in zip(shapes, U.structured_grads("spiked", shapes))]


def test_refresh_tc_spiked_spectrum_is_bf16_limited():
    # With a few singular values far above the rest, the bf16 rounding of the
    # dominant part is of the order of the small singular values, and NS5
    # amplifies those by ~3.4x per iteration.  That is a property of bf16
    # operands, not of the kernels: the CPU emulation of the format gives
    # 5-6e-2 on this input (tests/test_bf16_emulation.py).  The kernel must
    # stay within 1.5 x the emulated error; the fp32 check mode (parameters
    # stored as bf16 here) is two orders better.
    shapes = [(512, 1024)]
    fast = _structured_case("spiked", shapes, False)
    check = _structured_case("spiked", shapes, True)
    for e, bound in zip(fast, spiked_bounds(shapes)):
        assert e <= bound, (fast, bound)
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


def test_refresh_follows_parameters_that_move_on_a_live_handle():
    """The staged final update reaches the parameters through tensor maps kept
    in the workspace.  When the caller hands the same handle other parameter
    buffers, the maps are rewritten; the next refresh must use the new ones
    (and leave the old buffers alone), wide and tall."""
    shapes = [(256, 512), (512, 256), (1024, 2560)]
    cfg = U.oracle_cfg(K=1, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 31, "bf16", grad_std=1e-3, mom_std=1e-3)
    opt = B.PeriodicRowwiseMuon(shapes, cfg.K, cfg.beta, cfg.nesterov, cfg.lr, cfg.wd)
    A = [U.Guarded(w) for w in W]
    Bm = [U.Guarded(w) for w in W]
    g = [x.cuda() for x in G]
    mA = [x.cuda() for x in M]
    mB = [x.cuda() for x in M]
    opt.step([x.t for x in A], g, mA, 0)
    torch.cuda.synchronize()
    A_after = [x.t.clone() for x in A]
    opt.step([x.t for x in Bm], g, mB, 0)          # same handle, parameters elsewhere; A stays allocated
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for i, s in enumerate(shapes):
        assert A[i].intact() and Bm[i].intact()
        assert torch.equal(A[i].t, A_after[i]), f"{s}: the old parameter buffer was written again"
        assert torch.equal(Bm[i].t, A_after[i]), f"{s}: same inputs, same handle, other buffer: same bits"
        Wr, _ = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        w0 = U.to_np64(W[i])
        d_gpu = (1 - cfg.lr * cfg.wd) * w0 - U.to_np64(Bm[i].t)
        d_ref = (1 - cfg.lr * cfg.wd) * w0 - Wr
        # The update (~5e-3 * 1/sqrt(c) per element) is small against the half ulp of bf16
        # parameters of size ~2e-2, so the direction read back through them is coarse: the
        # parameters must agree closely, the recovered direction roughly.
        assert np.abs(U.to_np64(Bm[i].t) - Wr).max() <= 1e-3, s
        assert U.rel_fro(d_gpu, d_ref) <= 0.5, s
    opt.close()
