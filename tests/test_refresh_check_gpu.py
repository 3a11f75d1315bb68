"""GPU parity of the refresh branch (rho_t = 1) in fp32 check mode against
the fp64 oracle, plus whole trajectories of configuration 1."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from paper_2608_20818_b200.workloads import make_grad, make_momentum, make_param, workload
from tests import util as U

pytestmark = pytest.mark.gpu

SHAPES = [(256, 1024), (24, 40), (40, 24), (300, 520), (512, 256), (5, 5), (1, 9), (130, 1000), (768, 768)]


def _direction_case(shapes, io, check_mode, seed, nesterov=True, ns_ws=None, gram_span=2):
    """W = 0, lr = 1, wd = 0: the step writes -s * NS5 direction."""
    cfg = U.oracle_cfg(K=3, beta=0.95, nesterov=nesterov, lr=1.0, wd=0.0, scale_mode=0)
    W, G, M = U.make_inputs(shapes, seed, io, grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    Wg, Mg = U.gpu_step(shapes, W, G, M, 3, cfg, io, check_mode, ns_workspace_bytes=ns_ws, gram_span=gram_span)
    errs = []
    for i in range(len(shapes)):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 3, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {shapes[i]}")
        errs.append(U.rel_fro(Wg[i], Wr))
    return errs


@pytest.mark.parametrize("shape", SHAPES)
def test_refresh_check_mode_direction(shape):
    (err,) = _direction_case([shape], "fp32", True, seed=sum(shape))
    assert err <= 1e-4, err


def test_refresh_check_mode_groups_and_sub_batches():
    shapes = [(256, 512), (512, 256), (256, 512), (256, 256), (256, 512), (512, 256)]
    # cap small enough that the three 256x512 matrices are refreshed one at a time
    errs = _direction_case(shapes, "fp32", True, seed=3, ns_ws=1)
    assert max(errs) <= 1e-4, errs
    errs = _direction_case(shapes, "fp32", True, seed=3, nesterov=False)
    assert max(errs) <= 1e-4, errs


def test_refresh_full_update_bf16_io_check_mode():
    shapes = [(256, 1024), (1024, 256)]
    cfg = U.oracle_cfg(K=2, nesterov=True, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 11, "bf16", grad_std=1e-3, mom_std=1e-3)
    Wg, Mg = U.gpu_step(shapes, W, G, M, 2, cfg, "bf16", True)
    for i in range(2):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 2, cfg)
        U.assert_elementwise(Mg[i], Mr, False, "momentum")
        U.assert_elementwise(Wg[i], Wr, True, "param", rtol=2e-5)


def test_refresh_zero_matrix():
    shapes = [(64, 128)]
    cfg = U.oracle_cfg(K=1, lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 12, "fp32")
    G[0].zero_()
    M[0].zero_()
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, "fp32", True)
    np.testing.assert_allclose(Wg[0], (1 - 5e-5) * U.to_np64(W[0]), rtol=1e-6)
    assert not np.any(Mg[0])


def _config1_trajectory(check_mode, tol_dir):
    wl = workload(1)
    cfg = U.oracle_cfg(K=wl.K, beta=wl.beta, nesterov=wl.nesterov, lr=wl.lr, wd=wl.wd, gamma=wl.gamma)
    W0 = [make_param(wl, 0)]
    M0 = [make_momentum(wl, 0)]
    grads = [[make_grad(wl, 0, t)] for t in range(8)]
    opt = B.PeriodicRowwiseMuon(wl.shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma,
                                io_dtype="fp32", check_mode=check_mode)
    Wd, Md, Gd = W0[0].cuda(), M0[0].cuda(), torch.empty_like(W0[0], device="cuda")
    Wr, Mr = U.to_np64(W0[0]), U.to_np64(M0[0])
    refreshes = 0
    for t in range(8):
        Gd.copy_(grads[t][0])
        W_before = U.to_np64(Wd)
        opt.step([Wd], [Gd], [Md], t)
        torch.cuda.synchronize()
        refresh, _, _, _ = opt.plan(t)
        refreshes += refresh
        # oracle step from the oracle's own trajectory
        Mr_prev = Mr
        Wr, Mr = O.step_matrix(Wr, U.to_np64(grads[t][0]), Mr_prev, t, cfg)
        U.assert_elementwise(U.to_np64(Md), Mr, False, f"momentum t={t}")
        if refresh:
            # direction recovered from the update, compared in relative Frobenius norm
            Wo, _ = O.step_matrix(W_before, U.to_np64(grads[t][0]), Mr_prev, t, cfg)
            d_gpu = (1 - wl.lr * wl.wd) * W_before - U.to_np64(Wd)
            d_ref = (1 - wl.lr * wl.wd) * W_before - Wo
            assert U.rel_fro(d_gpu, d_ref) <= tol_dir
        if check_mode:
            U.assert_elementwise(U.to_np64(Wd), Wr, False, f"param t={t}")
    assert refreshes == 2 and opt.status() == B.PRM_OK
    opt.close()


def test_config1_eight_steps_check_mode():
    _config1_trajectory(True, 2e-4)


def test_resume_is_bit_identical():
    wl = workload(1)
    kw = dict(gamma=wl.gamma, io_dtype="fp32", check_mode=True)

    def run(split):
        W, M = make_param(wl, 0).cuda(), make_momentum(wl, 0).cuda()
        G = torch.empty_like(W)
        opt = B.PeriodicRowwiseMuon(wl.shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, **kw)
        for t in range(8):
            if t == split:
                opt.close()
                opt = B.PeriodicRowwiseMuon(wl.shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, **kw)
            G.copy_(make_grad(wl, 0, t))
            opt.step([W], [G], [M], t)
        torch.cuda.synchronize()
        opt.close()
        return W.cpu(), M.cpu()

    a, b = run(-1), run(4)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
