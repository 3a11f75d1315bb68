"""The Gram-space evaluation of the first three NS5 iterations (tensor-core
path, matrices with at least 1024 oriented rows and c >= 1.5 r) against the
fp64 oracle, which runs the five iterations as the paper prints them.  Both
evaluations are the same polynomial of the input in exact arithmetic; the
bound is the one of the tensor-core path: relative Frobenius error of the
direction at most 2e-2 per matrix."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from tests import util as U
from tests.test_refresh_check_gpu import _direction_case
from tests.test_refresh_tc_gpu import _structured_case, spiked_bounds

pytestmark = pytest.mark.gpu

TOL = 2e-2
# (shape, Gram-space iterations expected): oriented rows padded to >= 1024 and padded c >= 1.5 r
CASES = [((1024, 3072), 3), ((4096, 1024), 3), ((1024, 2048), 3), ((2048, 1024), 3), ((1100, 3000), 3), ((1024, 1536), 3), ((1280, 1792), 0),
         ((1024, 1024), 0), ((768, 3072), 0), ((1030, 2000), 3), ((3000, 1100), 3)]


@pytest.mark.parametrize("shape,iters", CASES)
def test_gramspace_direction_within_bound_and_eligibility(shape, iters):
    for mode, want in ((2, iters), (1, iters), (0, 0)):
        opt = B.PeriodicRowwiseMuon([shape], 1, gram_span=mode)
        assert opt.groups()[0]["gram_iters"] == want
        opt.close()
    errs = [_direction_case([shape], "bf16", False, seed=sum(shape), gram_span=mode)[0] for mode in (0, 1, 2)]
    assert max(errs) <= TOL, errs
    r, c = min(shape), max(shape)
    r_p, c_p = -(-r // 256) * 256, -(-c // 256) * 256
    if iters == 0:
        assert errs[0] == errs[1] == errs[2]
    elif c_p <= 2 * r_p:
        assert errs[1] == errs[2]          # the last Gram matrix is recomputed unless c > 2r


def test_gramspace_launch_classes_and_sub_batches():
    # (1024, 2560): c > 2r, so mode 2 takes the last Gram matrix from the one before it
    shapes = [(1024, 2048)] * 3 + [(2048, 1024)] * 2 + [(512, 1024)] + [(1024, 2560)]
    cfg = U.oracle_cfg(K=1, nesterov=True, lr=1.0, wd=0.0, scale_mode=0)
    W, G, M = U.make_inputs(shapes, 17, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    for mode in (1, 2):
        for ns_ws, sub_batches in ((None, (1, 1, 1, 1)), (1, (3, 2, 1, 1))):
            opt = B.PeriodicRowwiseMuon(shapes, 1, 0.95, True, 1.0, 0.0, scale_mode=0, ns_workspace_bytes=ns_ws,
                                        gram_span=mode)
            info = opt.groups()
            assert [g["gram_iters"] for g in info] == [3, 3, 0, 3]
            r, c = 1024.0, 2560.0
            assert info[3]["ns5_flop"] == (8 * r * r * c + 13 * r ** 3 if mode == 2 else 9 * r * r * c + 11 * r ** 3)
            assert info[0]["ns5_flop"] == 9 * r * r * 2048 + 11 * r ** 3
            assert info[2]["ns5_flop"] == 15 * 512.0 ** 2 * 1024 + 5 * 512.0 ** 3
            w = [x.cuda() for x in W]
            g = [x.cuda() for x in G]
            m = [x.cuda() for x in M]
            opt.profile(True)
            opt.step(w, g, m, 0)
            prof = opt.profile_read()
            torch.cuda.synchronize()
            assert opt.status() == B.PRM_OK
            n_gram = sub_batches[0] + sub_batches[1]          # sub-batches refreshed in Gram space
            n_printed = sub_batches[2]
            n_rec = 0
            if mode == 2:
                n_rec = sub_batches[3]                        # ... and with the last Gram matrix by recurrence
            else:
                n_gram += sub_batches[3]
            assert prof["gramspace"][1] == 6 * n_gram + 8 * n_rec
            assert prof["gram"][1] == 3 * n_gram + 5 * n_printed + 2 * n_rec
            assert prof["poly"][1] == 5 * (n_gram + n_printed + n_rec)
            assert prof["update"][1] == 2 * (n_gram + n_rec) + 4 * n_printed
            assert prof["update_final"][1] == n_gram + n_printed + n_rec
            for i, s in enumerate(shapes):
                Wr, _ = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
                assert U.rel_fro(U.to_np64(w[i]), Wr) <= TOL, (i, s)
            opt.close()


@pytest.mark.parametrize("kind", ["heavy_rows", "low_rank_mild"])
def test_gramspace_structured_inputs(kind):
    errs = _structured_case(kind, [(1024, 2048), (2048, 1024), (1024, 3072), (3072, 1024)], False)
    assert max(errs) <= TOL, errs


def test_gramspace_spiked_spectrum_within_the_emulated_format_error():
    shapes = [(1024, 2048), (1024, 3072)]
    errs = _structured_case("spiked", shapes, False)
    for e, bound in zip(errs, spiked_bounds(shapes)):
        assert e <= bound, (errs, bound)


def test_gramspace_is_reproducible_and_close_to_check_mode():
    shapes = [(1024, 2560), (2560, 1024)]
    cfg = U.oracle_cfg(K=2, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 29, "fp32", grad_std=1e-3, mom_std=1e-3)
    a = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", False)
    b = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", False)
    c = U.gpu_step(shapes, W, G, M, 2, cfg, "fp32", True)
    for i in range(2):
        assert np.array_equal(a[0][i], b[0][i]) and np.array_equal(a[1][i], b[1][i])
        w0 = U.to_np64(W[i])
        assert U.rel_fro((1 - 5e-5) * w0 - a[0][i], (1 - 5e-5) * w0 - c[0][i]) <= TOL


@pytest.mark.parametrize("io", ["bf16", "fp32"])
def test_gramspace_ragged_shapes_and_unaligned_columns(io):
    # columns not a multiple of 8 take the per-thread final update; fp32 parameters too
    shapes = [(1030, 2051), (2051, 1030), (1288, 3080), (1025, 2307)]
    opt = B.PeriodicRowwiseMuon(shapes, 1, io_dtype=io)
    assert [g["gram_iters"] for g in opt.groups()] == [3, 3, 3, 3]
    opt.close()
    errs = _direction_case(shapes, io, False, seed=77)
    assert max(errs) <= TOL, errs
