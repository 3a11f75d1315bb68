"""GPU parity of the tensor-core refresh with PRM_OPT_NS_SPLIT_INPUT = 1 (the NS5
input kept as two bf16 planes) against the fp64 oracle.

With the option every input kind stays inside the 2e-2 relative Frobenius bound of
the other refresh tests, the spiked spectrum included, whose error the default
(one bf16 plane) leaves at 5-6e-2 by the format alone; the kernel is also held to
1.5 x the error that the same arithmetic format gives in the numpy emulation.
Matrices with at most 768 oriented rows run in fp32 under the option, the larger
ones through the two-plane tensor-core products."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from tests import bf16_emulation as E
from tests import util as U
from tests.test_bf16_emulation import direction_input_of

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _case(kind, shapes, split, io="bf16", ns_ws=None, nesterov=True):
    cfg = U.oracle_cfg(K=1, nesterov=nesterov, lr=1.0, wd=0.0, scale_mode=0)
    W = [torch.zeros(s, dtype=torch.bfloat16 if io == "bf16" else torch.float32) for s in shapes]
    G = U.structured_grads(kind, shapes)
    if io == "fp32":
        G = [g.float() for g in G]
    M = [torch.zeros(s) for s in shapes]
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, io, False, ns_workspace_bytes=ns_ws, split_input=split)
    errs = []
    for i in range(len(shapes)):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {shapes[i]}")
        errs.append(U.rel_fro(Wg[i], Wr))
    return errs


SPIKED_SHAPES = [(1024, 3072), (1024, 1024), (2048, 1024), (1100, 1300), (1536, 1030), (512, 1024), (300, 520)]


def test_split_input_brings_the_spiked_spectrum_inside_the_general_bound():
    plain = _case("spiked", SPIKED_SHAPES, False)
    split = _case("spiked", SPIKED_SHAPES, True)
    for s, e0, e1 in zip(SPIKED_SHAPES, plain, split):
        assert e1 <= TOL, (s, e1)
        assert e0 >= 3e-2, (s, e0)                 # what the option is for
        assert e1 <= 0.4 * e0, (s, e0, e1)
        if min(s) <= 768:
            assert e1 <= 3e-3, (s, e1)             # fp32 recurrence, bf16 parameter store


def test_split_input_within_the_emulated_format_error():
    shapes = [(1024, 3072), (1280, 1280), (2048, 1024)]
    split = _case("spiked", shapes, True)
    for s, g, e in zip(shapes, U.structured_grads("spiked", shapes), split):
        Ut = direction_input_of(g, s)
        emu = E.emulated_error(Ut, E.library_schedule(s, split_input=True), split_input=True)
        assert e <= 1.5 * emu + 1e-3, (s, e, emu)


@pytest.mark.parametrize("kind", ["gauss", "heavy_rows", "low_rank_mild"])
def test_split_input_other_inputs_stay_inside_the_bound(kind):
    shapes = [(1024, 2560), (2560, 1024), (1024, 1024), (1100, 1300), (256, 256), (130, 1000)]
    errs = _case(kind, shapes, True)
    assert max(errs) <= TOL, errs


def test_split_input_groups_sub_batches_fp32_io_and_tiny_matrices():
    shapes = [(1024, 1536), (1536, 1024), (1024, 1536), (256, 256), (1024, 1536), (1536, 1024), (24, 40), (1024, 1024)]
    # workspace cap of one byte: every group is refreshed one matrix at a time
    for io in ("bf16", "fp32"):
        errs = _case("spiked", shapes, True, io=io, ns_ws=1)
        assert max(errs) <= TOL, (io, errs)
    errs = _case("spiked", shapes, True, nesterov=False)
    assert max(errs) <= TOL, errs


def test_split_input_is_reproducible_and_leaves_the_row_step_alone():
    shapes = [(1024, 1536), (1536, 1024)]
    cfg = U.oracle_cfg(K=2, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 9, "bf16", grad_std=1e-3, mom_std=1e-3)
    a = U.gpu_step(shapes, W, G, M, 2, cfg, "bf16", False, split_input=True)
    b = U.gpu_step(shapes, W, G, M, 2, cfg, "bf16", False, split_input=True)
    r0 = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, split_input=False)
    r1 = U.gpu_step(shapes, W, G, M, 1, cfg, "bf16", False, split_input=True)
    for i in range(2):
        assert np.array_equal(a[0][i], b[0][i]) and np.array_equal(a[1][i], b[1][i])
        assert np.array_equal(r0[0][i], r1[0][i]) and np.array_equal(r0[1][i], r1[1][i])


def test_split_input_multi_step_trajectory():
    """Eight steps at K = 4 (two refreshes, six row steps) on fresh gradients per step, fp32
    parameters: the momentum follows the oracle's element by element, and what the parameters
    moved by stays within the refresh bound of the oracle's trajectory (the row steps add no
    error of their own)."""
    shapes = [(1024, 1280), (1280, 1024), (256, 256)]
    cfg = U.oracle_cfg(K=4, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 21, "fp32", grad_std=1e-3, mom_std=1e-3)
    grads = {t: U.make_inputs(shapes, 100 + t, "fp32", grad_std=1e-3, mom_std=1e-3)[1] for t in range(8)}
    grads[0] = G
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, "fp32", False, steps=8, grads_fn=lambda t: grads[t], split_input=True)
    for i in range(len(shapes)):
        w, m = U.to_np64(W[i]), U.to_np64(M[i])
        for t in range(8):
            w, m = O.step_matrix(w, U.to_np64(grads[t][i]), m, t, cfg)
        U.assert_elementwise(Mg[i], m, False, f"momentum {shapes[i]}")
        assert U.rel_fro(U.to_np64(W[i]) - Wg[i], U.to_np64(W[i]) - w) <= TOL, shapes[i]
