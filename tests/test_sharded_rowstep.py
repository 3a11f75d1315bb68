"""Sharded tall RowNorm (Section 3.3 / Algorithm 2, non-refresh branch).

CPU: two gloo ranks run the orchestration (packing, asynchronous sum
all-reduce, wide matrices in the meantime, finish) with an oracle-arithmetic
backend and must reproduce the dense oracle step - the sharded-RowNorm
proposition.  GPU: the library's stats/apply entry points on uneven row shards
of one device, summed in place of the all-reduce, against the oracle and
against prm_step on the unsharded matrix."""

import math
import os

import numpy as np
import pytest
import torch
import torch.distributed as td
import torch.multiprocessing as mp

from oracle import prm_oracle as O
from paper_2608_20818_b200 import sharded as S
from tests import util as U

HP = dict(beta=0.95, nesterov=True, lr=5e-3, wd=0.01, gamma=0.15, eps_row=1e-8)


class OracleBackend:
    """stats/apply with the oracle's arithmetic on CPU tensors (fp64)."""

    def stats(self, grad, mom, out, stream):
        mt = O.momentum_update(mom.numpy(), grad.numpy(), HP["beta"])
        mom.copy_(torch.from_numpy(mt))
        u = O.direction_input(mt, grad.numpy(), HP["beta"], HP["nesterov"])
        out.copy_(torch.from_numpy((u * u).sum(axis=0)))

    scale_mode = 1

    def apply(self, param, grad, mom, colsumsq, global_rows, stream):
        scale = O.shape_scale(global_rows, param.shape[1], self.scale_mode)
        u = O.direction_input(mom.numpy(), grad.numpy(), HP["beta"], HP["nesterov"])
        nu = np.maximum(np.sqrt(colsumsq.numpy()), HP["eps_row"])
        w = (1 - HP["lr"] * HP["wd"]) * param.numpy() - HP["lr"] * scale * HP["gamma"] * u / nu
        param.copy_(torch.from_numpy(w))


def _dense_case(seed):
    rng = np.random.default_rng(seed)
    mats = []
    for (m, n) in [(24, 8), (40, 16)]:
        mats.append((rng.standard_normal((m, n)) * 0.02, rng.standard_normal((m, n)), rng.standard_normal((m, n)) * 0.1))
    return mats


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    td.init_process_group("gloo", rank=rank, world_size=world)
    mats = _dense_case(5)
    tall, called = [], []
    for (W, G, M) in mats:
        m = W.shape[0]
        lo, hi = (0, m // 3) if rank == 0 else (m // 3, m)        # uneven shards
        tall.append((torch.from_numpy(W[lo:hi].copy()), torch.from_numpy(G[lo:hi].copy()),
                     torch.from_numpy(M[lo:hi].copy()), m))
    tall64 = [(p.double(), g.double(), mm.double(), m) for (p, g, mm, m) in tall]

    S.sharded_row_step(tall64, lambda: called.append(1), OracleBackend(), stats_dtype=torch.float64)
    td.barrier()
    td.destroy_process_group()
    q.put((rank, [p.numpy() for (p, _, _, _) in tall64], [mm.numpy() for (_, _, mm, _) in tall64], called))


def test_two_gloo_ranks_reproduce_the_dense_step():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29700 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = {}
    for _ in range(2):
        r, W, M, called = q.get(timeout=120)
        out[r] = (W, M)
        assert called == [1]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = O.OracleConfig(K=4, **{k: HP[k] for k in ("beta", "nesterov", "lr", "wd", "gamma", "eps_row")})
    for i, (W, G, M) in enumerate(_dense_case(5)):
        Wr, Mr = O.step_matrix(W, G, M, 1, cfg)
        np.testing.assert_allclose(np.concatenate([out[0][0][i], out[1][0][i]]), Wr, rtol=1e-12)
        np.testing.assert_allclose(np.concatenate([out[0][1][i], out[1][1][i]]), Mr, rtol=1e-13)


def test_pack_offsets():
    assert S.pack_offsets([8, 16, 4]) == ([0, 8, 24], 28)
    assert S.pack_offsets([]) == ([], 0)


@pytest.mark.gpu
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_shards_on_one_gpu_match_oracle_and_prm_step(io):
    shape = (1000, 264)
    cuts = [0, 130, 131, 640, 1000]                                  # four uneven row shards
    cfg = U.oracle_cfg(K=4, **{k: HP[k] for k in ("beta", "nesterov", "lr", "wd", "gamma", "eps_row")})
    W, G, M = U.make_inputs([shape], 61, io)
    Wd, Gd, Md = W[0].cuda(), G[0].cuda(), M[0].cuda()
    be = S.CudaTallBackend(**HP)
    stream = torch.cuda.current_stream().cuda_stream
    parts = []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        out = torch.empty(shape[1], dtype=torch.float32, device="cuda")
        be.stats(Gd[lo:hi], Md[lo:hi], out, stream)
        parts.append(out)
    total = torch.stack(parts).sum(dim=0)                            # stands in for the sum all-reduce
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        be.apply(Wd[lo:hi], Gd[lo:hi], Md[lo:hi], total, shape[0], stream)
    torch.cuda.synchronize()
    Wr, Mr = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    U.assert_elementwise(U.to_np64(Md), Mr, False, "momentum")
    U.assert_elementwise(U.to_np64(Wd), Wr, io == "bf16", "param")
    # one rank, one shard, through the orchestration: same as prm_step
    Wg, Mg = U.gpu_step([shape], W, G, M, 1, cfg, io, True)
    W2, G2, M2 = W[0].cuda(), G[0].cuda(), M[0].cuda()
    S.sharded_row_step([(W2, G2, M2, shape[0])], None, be, stream=stream)
    torch.cuda.synchronize()
    U.assert_elementwise(U.to_np64(W2), Wg[0], io == "bf16", "param vs prm_step")
    assert np.array_equal(U.to_np64(M2), Mg[0])


@pytest.mark.gpu
@pytest.mark.parametrize("scale_mode", [0, 2])
def test_sharded_row_step_and_refresh_follow_the_scale_mode(scale_mode):
    """Both branches of the sharded execution take s(W) from the same option:
    the row step through the backend's scale mode, the refresh through the
    handle's."""
    from paper_2608_20818_b200 import binding as B
    shape = (1000, 264)
    cfg = U.oracle_cfg(K=2, scale_mode=scale_mode, **{k: HP[k] for k in ("beta", "nesterov", "lr", "wd", "gamma", "eps_row")})
    assert B.prm_shape_scale(scale_mode, *shape) == pytest.approx(O.shape_scale(shape[0], shape[1], scale_mode), rel=1e-7)
    W, G, M = U.make_inputs([shape], 62, "fp32", grad_std=1e-3, mom_std=1e-3)
    stream = torch.cuda.current_stream().cuda_stream
    # row step (t = 1) on one shard that is the whole matrix
    be = S.CudaTallBackend(scale_mode=scale_mode, **HP)
    W2, G2, M2 = W[0].cuda(), G[0].cuda(), M[0].cuda()
    S.sharded_row_step([(W2, G2, M2, shape[0])], None, be, stream=stream)
    torch.cuda.synchronize()
    Wr, Mr = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 1, cfg)
    U.assert_elementwise(U.to_np64(W2), Wr, False, f"row step, scale mode {scale_mode}")
    # refresh (t = 0) through the bucketed path with one rank, fp32 check mode
    opt = B.PeriodicRowwiseMuon([shape], cfg.K, cfg.beta, cfg.nesterov, cfg.lr, cfg.wd, scale_mode=scale_mode,
                                io_dtype="fp32", check_mode=True)
    W3, G3, M3 = W[0].cuda(), G[0].cuda(), M[0].cuda()
    S.bucketed_refresh_step([shape], [W3], [G3], [M3], S.CudaRefreshBackend(opt, cfg.beta, cfg.nesterov))
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    Wr0, _ = O.step_matrix(U.to_np64(W[0]), U.to_np64(G[0]), U.to_np64(M[0]), 0, cfg)
    w0 = U.to_np64(W[0])
    d_gpu = (1 - cfg.lr * cfg.wd) * w0 - U.to_np64(W3)
    d_ref = (1 - cfg.lr * cfg.wd) * w0 - Wr0
    # the gathered payload is bf16 (2^-9 per element), NS5 itself runs in fp32 here
    assert U.rel_fro(d_gpu, d_ref) <= 1e-2, U.rel_fro(d_gpu, d_ref)
    opt.close()
