"""The allocation-free row step for tall matrices against the oracle and the
regular path.

Some users of this library cannot allocate device memory at all (their host
process has already handed the whole GPU to its own memory pool, or they run
in a loop that must not take the device-wide stall of cudaMalloc), so they
cannot attach the workspace that `prm_step` needs for the column norms of
tall matrices.  `prm_rowstep_tall_noalloc` serves them from a fixed array
inside the library.  This file checks that it computes what the oracle and
`prm_step` compute, on calls in a row that share that array, at the largest
size the array holds, and that it refuses matrices too large for it.  It is
collected last on purpose.
"""

import gc
import math

import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from tests import util as U


def _call(w, g, m, cfg, shape):
    B.prm_rowstep_tall_noalloc(w, g, m, beta=cfg.beta, nesterov=cfg.nesterov, lr=cfg.lr, wd=cfg.wd,
                               gamma=cfg.gamma, eps_row=cfg.eps_row,
                               scale=O.shape_scale(shape[0], shape[1], cfg.scale_mode))


def _both_paths(shape, io, nesterov, seed, check_free_memory):
    cfg = U.oracle_cfg(K=4, beta=0.95, nesterov=nesterov, lr=5e-3, wd=0.01, gamma=0.15, eps_row=1e-8)
    W, G, M = U.make_inputs([shape], seed, io)
    # existing entry point (workspace allocated by torch)
    W_ref, M_ref = U.gpu_step([shape], W, G, M, t=1, cfg=cfg, io=io, check_mode=True)
    # the oracle
    W_orc, M_orc = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    # new entry point: no workspace, no handle
    w, g, m = U.Guarded(W[0]), U.Guarded(G[0]), U.Guarded(M[0])
    # Nothing may be allocated by the call: not through torch (its allocator's counter) and not
    # behind its back (the driver's free-memory figure; meaningful from the second call on, when
    # the library's built-in array has been materialised).  Garbage of earlier tests is collected
    # first so that only the call is measured.
    gc.collect()
    torch.cuda.synchronize()
    gc.disable()
    try:
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]
        _call(w.t, g.t, m.t, cfg, shape)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        if check_free_memory:
            assert torch.cuda.mem_get_info()[0] >= free_before
    finally:
        gc.enable()
    assert w.intact() and g.intact() and m.intact()
    assert torch.equal(g.t.cpu(), G[0])
    for what, Mx, Wx in (("prm_step", M_ref[0], W_ref[0]), ("oracle", M_orc, W_orc)):
        U.assert_elementwise(U.to_np64(m.t), Mx, False, f"momentum {shape} against {what}")
        U.assert_elementwise(U.to_np64(w.t), Wx, io == "bf16", f"param {shape} against {what}")


@pytest.mark.gpu
def test_no_alloc_matches_oracle_and_step_on_calls_in_a_row():
    # the second call is smaller and of the other storage type, so it runs on
    # an array that still holds the first call's partial sums
    _both_paths((2048, 512), "bf16", True, seed=21, check_free_memory=False)
    _both_paths((1000, 264), "fp32", False, seed=22, check_free_memory=True)
    _both_paths((2048, 512), "bf16", True, seed=23, check_free_memory=True)


@pytest.mark.gpu
def test_no_alloc_at_the_largest_size_the_array_holds():
    # (ceil(rows/128) + 1) * cols = 1023 + 1 blocks x 1024 columns = 2^20 floats: the last entry of the array is used
    shape = (130944, 1024)
    cfg = U.oracle_cfg(K=4, beta=0.95, nesterov=True, lr=5e-3, wd=0.01, gamma=0.15, eps_row=1e-8)
    W, G, M = U.make_inputs([shape], 24, "bf16")
    W_orc, M_orc = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    w, g, m = U.Guarded(W[0]), U.Guarded(G[0]), U.Guarded(M[0])
    _call(w.t, g.t, m.t, cfg, shape)
    torch.cuda.synchronize()
    assert w.intact() and g.intact() and m.intact()
    U.assert_elementwise(U.to_np64(m.t), M_orc, False, "momentum at the size limit")
    U.assert_elementwise(U.to_np64(w.t), W_orc, True, "param at the size limit")
    # one more row block does not fit
    too_big = (130945, 1024)
    p2 = torch.zeros(too_big, dtype=torch.bfloat16, device="cuda")
    m2 = torch.zeros(too_big, device="cuda")
    with pytest.raises(B.PrmError) as e:
        B.prm_rowstep_tall_noalloc(p2, p2.clone(), m2, beta=0.95, nesterov=True, lr=1e-3, wd=0.0, gamma=0.15,
                                   eps_row=1e-8, scale=1.0)
    assert e.value.code == B.PRM_ERR_WORKSPACE and "scratch" in str(e.value)


@pytest.mark.gpu
def test_no_alloc_refuses_what_does_not_fit_or_is_not_tall():
    big = (300000, 512)          # (ceil(rows/128)+1)*cols = 1.2M floats > 1M
    p = torch.zeros(big, dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(big, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(big, device="cuda")
    with pytest.raises(B.PrmError) as e:
        B.prm_rowstep_tall_noalloc(p, g, m, beta=0.95, nesterov=True, lr=1e-3, wd=0.0, gamma=0.15, eps_row=1e-8,
                                   scale=1.0)
    assert e.value.code == B.PRM_ERR_WORKSPACE and "scratch" in str(e.value)
    del p, g, m
    p = torch.zeros(8, 8, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(8, 8, device="cuda")
    with pytest.raises(B.PrmError) as e:
        B.prm_rowstep_tall_noalloc(p, p.clone(), m, beta=0.95, nesterov=True, lr=1e-3, wd=0.0, gamma=0.15,
                                   eps_row=1e-8, scale=1.0)
    assert e.value.code == B.PRM_ERR_SHAPE
    torch.cuda.synchronize()
    assert not p.any() and not m.any()


def test_no_alloc_binding_rejects_mismatched_tensors_before_any_launch():
    """The wrapper hands raw pointers to the kernels, so it must refuse tensors
    whose dtype, shape or layout is not what the kernels assume.  Runs without
    a GPU: every check comes before the C call."""
    kw = dict(beta=0.95, nesterov=True, lr=1e-3, wd=0.0, gamma=0.15, eps_row=1e-8, scale=1.0)
    p = torch.zeros(64, 16, dtype=torch.bfloat16)
    g = torch.zeros(64, 16, dtype=torch.bfloat16)
    m = torch.zeros(64, 16)
    with pytest.raises(TypeError):
        B.prm_rowstep_tall_noalloc(p, g.float(), m, **kw)              # gradient dtype differs
    with pytest.raises(TypeError):
        B.prm_rowstep_tall_noalloc(p, g, m.to(torch.bfloat16), **kw)   # momentum must be fp32
    with pytest.raises(TypeError):
        B.prm_rowstep_tall_noalloc(p.half(), g.half(), m, **kw)        # unsupported storage type
    with pytest.raises(ValueError):
        B.prm_rowstep_tall_noalloc(p, g, m[:32], **kw)                 # half-size momentum
    with pytest.raises(ValueError):
        B.prm_rowstep_tall_noalloc(p, g[:, :8], m, **kw)               # shape mismatch
    with pytest.raises(ValueError):
        B.prm_rowstep_tall_noalloc(p, g, torch.zeros(16, 64).t(), **kw)   # non-contiguous view
    with pytest.raises(ValueError):
        B.prm_rowstep_tall_noalloc(p.view(-1), g.view(-1), m.view(-1), **kw)   # not a matrix
    with pytest.raises(ValueError):
        B.prm_rowstep_tall_noalloc(p, g, m, **kw)                      # not on a CUDA device
