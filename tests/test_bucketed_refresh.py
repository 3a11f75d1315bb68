"""Refresh over row shards (Section 3.3; Algorithm 2 lines 1-7; appendix
"Idealized overlap model").

CPU: the planning functions of the C ABI against the oracle's and against what
fixes them independently (torch.chunk, an event simulation of the two-stage
pipeline, the invariants of a bucket plan); the oracle's shard-wise refresh
against its dense step; two gloo ranks running the orchestration with an
oracle-arithmetic backend against the dense oracle step.
GPU: the ranks of a world of 1, 2 or 3 emulated one after the other on one
device (the gathered buffer is the concatenation of the ranks' segments, which
is what an all-gather delivers), against the oracle and against prm_step on the
unsharded matrices."""

import os

import numpy as np
import pytest
import torch
import torch.distributed as td
import torch.multiprocessing as mp

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B
from paper_2608_20818_b200 import sharded as S
from paper_2608_20818_b200.workloads import workload
from tests import util as U


# ------------------------------------------------------------------ planning
def test_shard_rows_is_torch_chunk():
    for rows in list(range(1, 41)) + [4096, 16384, 5121]:
        for world in range(1, 10):
            chunks = torch.chunk(torch.arange(rows), world)
            for rank in range(world):
                want = (int(chunks[rank][0]), len(chunks[rank])) if rank < len(chunks) else (rows, 0)
                assert O.shard_rows(rows, world, rank) == want
                assert B.prm_shard_rows(rows, world, rank) == want
    with pytest.raises(B.PrmError):
        B.prm_shard_rows(8, 2, 2)


def _check_plan(shapes, world, cap, plan):
    bucket_of_mat, offsets, segments = plan
    n = len(shapes)
    assert len(bucket_of_mat) == len(offsets) == n
    # the walk: shape groups in order of first appearance, given order inside a group
    first = {}
    for i, sh in enumerate(shapes):
        first.setdefault(tuple(sh), i)
    walk = sorted(range(n), key=lambda i: (first[tuple(shapes[i])], i))
    ids = [bucket_of_mat[i] for i in walk]
    assert ids[0] == 0 and all(b1 - b0 in (0, 1) for b0, b1 in zip(ids, ids[1:]))
    assert len(segments) == ids[-1] + 1
    need = lambda i: -(-(-(-shapes[i][0] // world) * shapes[i][1]) // 8) * 8
    for l, seg in enumerate(segments):
        members = [i for i in walk if bucket_of_mat[i] == l]
        assert members, "empty bucket"
        end = 0
        for i in members:                      # slots in walk order, disjoint, 16-byte aligned, large enough
            assert offsets[i] == end and offsets[i] % 8 == 0
            end = offsets[i] + need(i)
        assert end == seg
        assert seg * 2 * world <= cap or len(members) == 1
        if l + 1 < len(segments):              # greedy: the next matrix would not have fitted
            nxt = [i for i in walk if bucket_of_mat[i] == l + 1][0]
            assert (seg + need(nxt)) * 2 * world > cap


def test_bucket_plan_matches_oracle_and_invariants():
    cases = [([(10, 8), (7, 3), (64, 64), (5, 5), (1, 9)], 3, 400),
             ([(10, 8)], 1, 1),
             (workload(4).shapes, 8, 240 << 20),
             (workload(2).shapes, 4, 64 << 20),
             (workload(5, 2).shapes, 7, 1 << 30)]
    for shapes, world, cap in cases:
        shapes = [tuple(s) for s in shapes]
        want = O.bucket_plan(shapes, world, cap)
        got = B.prm_bucket_plan(shapes, world, cap)
        assert got == tuple(want) or list(got) == list(want)
        _check_plan(shapes, world, cap, got)
    # the 9B-class set over 8 ranks in 240 MiB buckets: every bucket holds matrices of one shape
    shapes4 = [tuple(s) for s in workload(4).shapes]
    b, _, seg = B.prm_bucket_plan(shapes4, 8, 240 << 20)
    assert len(seg) > 42 and max(seg) * 16 <= 240 << 20 + 1
    mixed = sum(1 for l in range(len(seg)) if len({shapes4[i] for i in range(len(shapes4)) if b[i] == l}) > 1)
    assert mixed <= 4                          # only where one shape group ends and the next begins


def _simulate_pipeline(a, c):
    """Event simulation: the all-gather of bucket l+1 is launched when the
    compute of bucket l starts; compute l starts when its gather and compute
    l-1 are done."""
    n = len(a)
    gather_done = [0.0] * n
    compute_done = [0.0] * n
    gather_done[0] = a[0]
    busy_comm = 0.0
    for l in range(n):
        start = max(gather_done[l], compute_done[l - 1] if l else 0.0)
        if l:
            busy_comm += max(0.0, gather_done[l] - compute_done[l - 1])
        if l + 1 < n:
            gather_done[l + 1] = start + a[l + 1]
        compute_done[l] = start + c[l]
    return compute_done[-1], a[0] + busy_comm


def test_pipeline_model_against_event_simulation_and_closed_forms():
    rng = np.random.default_rng(3)
    for n in (1, 2, 3, 7, 20):
        for _ in range(20):
            a = rng.uniform(0, 5, n).tolist()
            c = rng.uniform(0, 5, n).tolist()
            want = _simulate_pipeline(a, c)
            for got in (O.pipeline_time(a, c), B.prm_pipeline_model(a, c)):
                assert got[0] == pytest.approx(want[0], rel=1e-12)
                assert got[1] == pytest.approx(want[1], rel=1e-12, abs=1e-12)
    # closed forms
    assert B.prm_pipeline_model([2.0], [3.0]) == (5.0, 2.0)
    assert B.prm_pipeline_model([1, 1, 1, 1], [4, 4, 4, 4]) == (17.0, 1.0)        # communication hidden
    assert B.prm_pipeline_model([4, 4, 4, 4], [1, 1, 1, 1]) == (17.0, 13.0)       # communication bound
    assert B.prm_pipeline_model([0, 0, 0], [1, 2, 3]) == (6.0, 0.0)
    assert B.prm_pipeline_model([1, 2, 3], [0, 0, 0]) == (6.0, 6.0)
    assert B.prm_pipeline_model([1, 2, 3], [2, 2, 2]) == (8.0, 2.0)               # worked by hand


def _split(x, world):
    return [x[slice(*(lambda lo_n: (lo_n[0], lo_n[0] + lo_n[1]))(O.shard_rows(x.shape[0], world, q)))] for q in range(world)]


def test_oracle_refresh_from_shards_equals_dense_step():
    rng = np.random.default_rng(11)
    cfg = O.OracleConfig(K=2, beta=0.9, nesterov=True, lr=3e-3, wd=0.02, scale_mode=1)
    for (m, n) in [(12, 20), (20, 12), (7, 7), (5, 16)]:
        W, G, M = rng.standard_normal((m, n)) * 0.02, rng.standard_normal((m, n)), rng.standard_normal((m, n)) * 0.1
        Wd, Md = O.step_matrix(W, G, M, 0, cfg)
        for world in (1, 2, 3, 6):
            Ws, Ms = O.refresh_from_shards(_split(W, world), _split(G, world), _split(M, world), cfg)
            np.testing.assert_allclose(np.concatenate(Ws), Wd, rtol=1e-12, atol=1e-15)
            np.testing.assert_allclose(np.concatenate(Ms), Md, rtol=1e-15)


# --------------------------------------------------- orchestration on CPU ranks
CFG = dict(K=1, beta=0.95, nesterov=True, lr=5e-3, wd=0.01, scale_mode=1)
SHAPES_CPU = [(24, 40), (40, 24), (9, 16), (24, 40), (16, 16), (30, 8)]


class OracleRefreshBackend:
    """pack / refresh with the oracle's arithmetic on CPU tensors (fp64 payload)."""

    payload_dtype = torch.float64

    def __init__(self, shapes, cfg):
        self.shapes, self.cfg = shapes, cfg

    def plan(self, shapes, world, bucket_bytes):
        return O.bucket_plan(shapes, world, bucket_bytes)

    def pack(self, grad, mom, cols, reserved, out, stream):
        mt = O.momentum_update(mom.numpy(), grad.numpy(), self.cfg.beta)
        mom.copy_(torch.from_numpy(mt))
        u = O.direction_input(mt, grad.numpy(), self.cfg.beta, self.cfg.nesterov)
        out.zero_()
        out[:u.size] = torch.from_numpy(u.reshape(-1))

    def refresh(self, mats, gathered, segment_elems, offsets, world, rank, param_shards, stream):
        cfg = self.cfg
        for i, off, p in zip(mats, offsets, param_shards):
            rows, cols = self.shapes[i]
            parts = []
            for q in range(world):                            # rebuild the full matrix from the segments
                _, cnt = O.shard_rows(rows, world, q)
                seg = gathered[q * segment_elems + off: q * segment_elems + off + cnt * cols]
                parts.append(seg.numpy().reshape(cnt, cols))
            u = np.concatenate(parts, axis=0)
            d = O.shape_scale(rows, cols, cfg.scale_mode) * O.direction(u, True, cfg)
            lo, cnt = O.shard_rows(rows, world, rank)
            p.copy_(torch.from_numpy((1 - cfg.lr * cfg.wd) * p.numpy() - cfg.lr * d[lo:lo + cnt]))


def _dense_inputs(seed):
    rng = np.random.default_rng(seed)
    return [(rng.standard_normal(s) * 0.02, rng.standard_normal(s), rng.standard_normal(s) * 0.1) for s in SHAPES_CPU]


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    td.init_process_group("gloo", rank=rank, world_size=world)
    cfg = O.OracleConfig(**CFG)
    mats = _dense_inputs(7)
    shard = lambda x: torch.from_numpy(_split(x, world)[rank].copy())
    P = [shard(W) for (W, _, _) in mats]
    G = [shard(Gm) for (_, Gm, _) in mats]
    M = [shard(Mm) for (_, _, Mm) in mats]
    trace = []
    # small cap: several buckets, the largest matrices alone in theirs
    plan = S.bucketed_refresh_step(SHAPES_CPU, P, G, M, OracleRefreshBackend(SHAPES_CPU, cfg), bucket_bytes=2500,
                                   trace=trace)
    td.barrier()
    q.put((rank, [p.numpy() for p in P], [m.numpy() for m in M], trace, plan))
    td.destroy_process_group()


def test_bucketed_refresh_two_gloo_ranks_equals_dense_oracle():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=180) for _ in range(world)], key=lambda t: t[0])
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    cfg = O.OracleConfig(**CFG)
    mats = _dense_inputs(7)
    for i, (W, G, M) in enumerate(mats):
        Wd, Md = O.step_matrix(W, G, M, 0, cfg)
        np.testing.assert_allclose(np.concatenate([got[r][1][i] for r in range(world)]), Wd, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(np.concatenate([got[r][2][i] for r in range(world)]), Md, rtol=1e-15)
    # Algorithm 2 lines 2-6: first gather up front, then gather l+1 is issued before refresh l
    n_buckets = len(got[0][4][2])
    assert n_buckets >= 3
    want = [("gather", 0)]
    for l in range(n_buckets):
        if l + 1 < n_buckets:
            want.append(("gather", l + 1))
        want.append(("refresh", l))
    assert got[0][3] == want and got[1][3] == want


def test_bucketed_refresh_needs_a_process_group_for_world_above_one():
    with pytest.raises(ValueError):
        S.bucketed_refresh_step([(4, 4)], [torch.zeros(2, 4)], [torch.zeros(2, 4)], [torch.zeros(2, 4)],
                                OracleRefreshBackend([(4, 4)], O.OracleConfig(**CFG)), world=2, rank=0)


# ------------------------------------------------------------------- on a GPU
def _emulate_world(shapes, W, G, M, world, cfg, io, check_mode, bucket_bytes, in_place=False, split_input=False):
    """All ranks of `world` one after the other on one device.  Returns full
    (W_new, M_new) as fp64 numpy, shards concatenated."""
    dev = "cuda"
    opt = B.PeriodicRowwiseMuon(shapes, cfg.K, cfg.beta, cfg.nesterov, cfg.lr, cfg.wd, gamma=cfg.gamma,
                                eps_ns=cfg.eps_ns, scale_mode=cfg.scale_mode, io_dtype=io, check_mode=check_mode,
                                split_input=split_input)
    bucket_of_mat, offsets, segments = B.prm_bucket_plan(shapes, world, bucket_bytes)
    n = len(shapes)
    cut = lambda x, q, rows: x[slice(*(lambda lo_n: (lo_n[0], lo_n[0] + lo_n[1]))(B.prm_shard_rows(rows, world, q)))]
    Ws = [[U.Guarded(cut(W[i], q, shapes[i][0]).contiguous()) for i in range(n)] for q in range(world)]
    Gs = [[U.Guarded(cut(G[i], q, shapes[i][0]).contiguous()) for i in range(n)] for q in range(world)]
    Ms = [[U.Guarded(cut(M[i], q, shapes[i][0]).contiguous()) for i in range(n)] for q in range(world)]
    stream = torch.cuda.current_stream().cuda_stream
    for l, seg in enumerate(segments):
        members = [i for i in range(n) if bucket_of_mat[i] == l]
        sends = []
        for q in range(world):
            send = torch.full((seg,), float("nan"), dtype=torch.bfloat16, device=dev)   # every element must be written
            for i in members:
                rows, cols = shapes[i]
                reserved = -(-(-(-rows // world) * cols) // 8) * 8
                B.prm_shard_momentum_pack(Gs[q][i].t, Ms[q][i].t, cols, reserved, cfg.beta, cfg.nesterov,
                                          send[offsets[i]:].data_ptr())
            sends.append(send)
        gathered = torch.cat(sends)                                # what an all-gather delivers
        assert not torch.isnan(gathered.float()).any()
        for q in range(world):
            ptrs = [Ws[q][i].t.data_ptr() if Ws[q][i].t.numel() else 0 for i in members]
            if in_place:        # no gathered copy: every rank's segment is read where it was packed
                B.prm_refresh_segments(opt.h, members, [x.data_ptr() for x in sends], seg,
                                       [offsets[i] for i in members], world, q, ptrs, stream)
            else:
                B.prm_refresh_gathered(opt.h, members, gathered.data_ptr(), seg, [offsets[i] for i in members], world,
                                       q, ptrs, stream)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for q in range(world):
        for x in Ws[q] + Gs[q] + Ms[q]:
            assert x.intact(), "write outside a shard"
    opt.close()
    Wn = [np.concatenate([U.to_np64(Ws[q][i].t) for q in range(world)]) for i in range(n)]
    Mn = [np.concatenate([U.to_np64(Ms[q][i].t) for q in range(world)]) for i in range(n)]
    return Wn, Mn


GPU_SHAPES = [(70, 40), (40, 72), (300, 520), (512, 256), (70, 40), (33, 17), (256, 256)]


@pytest.mark.gpu
@pytest.mark.parametrize("world", [1, 2, 3])
def test_sharded_refresh_check_mode_exact_payload(world):
    # beta = 1/2, no Nesterov, inputs on a grid of 1/16: the direction input is exactly
    # representable in bf16, so the gathered payload loses nothing and the fp32 check mode
    # must agree with the fp64 oracle as closely as on one GPU.
    cfg = U.oracle_cfg(K=1, beta=0.5, nesterov=False, lr=1.0, wd=0.0, scale_mode=1)
    g = torch.Generator().manual_seed(100 + world)
    W = [torch.zeros(s) for s in GPU_SHAPES]
    G = [torch.randint(-8, 9, s, generator=g).float() / 16 for s in GPU_SHAPES]
    M = [torch.randint(-8, 9, s, generator=g).float() / 16 for s in GPU_SHAPES]
    Wn, Mn = _emulate_world(GPU_SHAPES, W, G, M, world, cfg, "fp32", True, bucket_bytes=300000)
    for i, s in enumerate(GPU_SHAPES):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        U.assert_elementwise(Mn[i], Mr, False, f"momentum {s}")
        assert U.rel_fro(Wn[i], Wr) <= 1e-4, (s, U.rel_fro(Wn[i], Wr))


@pytest.mark.gpu
@pytest.mark.parametrize("io", ["bf16", "fp32"])
def test_sharded_refresh_tensor_cores_against_oracle_and_across_world_sizes(io):
    shapes = GPU_SHAPES + [(1024, 2048), (2048, 1024), (1100, 1992)]       # the last three use the Gram-space iterations
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=1.0, wd=0.0, scale_mode=1)
    W, G, M = U.make_inputs(shapes, 40, io, grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    Wu, Mu = U.gpu_step(shapes, W, G, M, 0, cfg, io, False)
    first = None
    for world, cap in ((1, 3 << 20), (2, 3 << 20), (3, 1 << 20), (5, 64 << 20)):
        Wn, Mn = _emulate_world(shapes, W, G, M, world, cfg, io, False, bucket_bytes=cap)
        if first is None:
            first = Wn
        for i, s in enumerate(shapes):
            Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
            U.assert_elementwise(Mn[i], Mr, False, f"momentum {s}")
            assert np.array_equal(Mn[i], Mu[i]), "momentum must not depend on the sharding"
            assert U.rel_fro(Wn[i], Wr) <= 2e-2, (s, world, U.rel_fro(Wn[i], Wr))
            # The rebuilt NS5 input, its norm and every product are the same for any number of
            # ranks and any bucketing, so the result must not change by a single bit.
            assert np.array_equal(Wn[i], first[i]), (s, world)
            # Against the unsharded step only the Frobenius norm differs (summed before instead of
            # after the bf16 rounding of U, ~1e-5 relative); the bf16 roundings of the recurrence then
            # fall differently, which moves the result by a good part of its own rounding noise.
            assert U.rel_fro(Wn[i], Wu[i]) <= 2e-2, (s, U.rel_fro(Wn[i], Wu[i]))


@pytest.mark.gpu
def test_sharded_refresh_on_a_handle_with_split_input():
    """PRM_OPT_NS_SPLIT_INPUT changes the workspace layout (a second plane of X_0), the order of
    evaluation (Gram space for every matrix from 1024 padded rows on) and sends smaller matrices
    to fp32.  The sharded refresh, whose bf16 payload has no second plane, runs on the same handle:
    one plane, the same layout and schedule."""
    shapes = GPU_SHAPES + [(1024, 2048), (2048, 1024), (1100, 1100)]
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=1.0, wd=0.0, scale_mode=1)
    W, G, M = U.make_inputs(shapes, 41, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    first = None
    for world, cap in ((1, 3 << 20), (3, 1 << 20)):
        Wn, Mn = _emulate_world(shapes, W, G, M, world, cfg, "bf16", False, bucket_bytes=cap, split_input=True)
        first = first or Wn
        for i, s in enumerate(shapes):
            Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
            U.assert_elementwise(Mn[i], Mr, False, f"momentum {s}")
            # below 1024 padded rows: fp32 recurrence on the bf16 payload (its rounding, 2^-9 per
            # element, is what is left); above: the tensor-core path as without the option
            assert U.rel_fro(Wn[i], Wr) <= (6e-3 if min(s) <= 768 else 2e-2), (s, world, U.rel_fro(Wn[i], Wr))
            assert np.array_equal(Wn[i], first[i]), (s, world)


@pytest.mark.gpu
def test_refresh_segments_reads_every_rank_in_place():
    shapes = GPU_SHAPES + [(1024, 2560)]
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=5e-3, wd=0.01, scale_mode=1)
    W, G, M = U.make_inputs(shapes, 61, "bf16", grad_std=1e-3, mom_std=1e-3)
    for world in (1, 3):
        a = _emulate_world(shapes, W, G, M, world, cfg, "bf16", False, bucket_bytes=2 << 20)
        b = _emulate_world(shapes, W, G, M, world, cfg, "bf16", False, bucket_bytes=2 << 20, in_place=True)
        for i in range(len(shapes)):
            assert np.array_equal(a[0][i], b[0][i]) and np.array_equal(a[1][i], b[1][i])


@pytest.mark.gpu
def test_p2p_exchange_through_symmetric_memory_one_rank():
    import subprocess
    import sys
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "p2p_refresh_worker.py")
    r = subprocess.run([sys.executable, worker], env=env, capture_output=True, text=True, timeout=600)
    last = (r.stdout.strip().splitlines() or [""])[-1]
    if last.startswith("SKIP"):
        pytest.skip("torch symmetric memory is not usable here: " + last)
    assert r.returncode == 0 and last == "OK", (r.stdout[-500:], r.stderr[-1500:])


@pytest.mark.gpu
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_sharded_refresh_full_update_with_decay(io):
    shapes = [(512, 1024), (1024, 512), (300, 520)]
    cfg = U.oracle_cfg(K=1, beta=0.95, nesterov=True, lr=5e-3, wd=0.01, scale_mode=1)
    W, G, M = U.make_inputs(shapes, 77, io, grad_std=1e-3, mom_std=1e-3)
    Wn, _ = _emulate_world(shapes, W, G, M, 2, cfg, io, True, bucket_bytes=1 << 20)
    for i, s in enumerate(shapes):
        w0 = U.to_np64(W[i])
        Wr, _ = O.step_matrix(w0, U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        step_ref = (1 - cfg.lr * cfg.wd) * w0 - Wr
        if io == "fp32":
            # fp32 NS5 on a payload rounded to bf16: the direction moves by a few 1e-3 of itself
            step_got = (1 - cfg.lr * cfg.wd) * w0 - Wn[i]
            assert U.rel_fro(step_got, step_ref) <= 5e-3
            assert np.abs(Wn[i] - Wr).max() <= 1e-2 * np.abs(step_ref).max()
        else:
            # one bf16 store on top: never more than one ulp away, and only where the small
            # change of the direction crosses a rounding boundary
            ulp = 2 * U.bf16_half_ulp(Wr)
            slack = 1e-2 * np.abs(step_ref).max()          # the change of the direction itself
            diff = np.abs(Wn[i] - Wr)
            assert (diff <= ulp * (1 + 1e-3) + slack).all()
            assert (diff > 0.5 * ulp * (1 + 1e-3) + slack).mean() <= 0.03


@pytest.mark.gpu
def test_bucketed_refresh_step_single_rank_matches_prm_step():
    wl = workload(2, 1)
    shapes = [tuple(s) for s in wl.shapes]
    cfg = U.oracle_cfg(K=wl.K, beta=wl.beta, nesterov=wl.nesterov, lr=wl.lr, wd=wl.wd, gamma=wl.gamma)
    W, G, M = U.make_inputs(shapes, 5, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()                   # the step then writes -lr*s*D with the full relative precision of bf16
    Wu, Mu = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", False)
    opt = B.PeriodicRowwiseMuon(shapes, wl.K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma)
    P = [w.cuda() for w in W]
    Gd = [g.cuda() for g in G]
    Md = [m.cuda() for m in M]
    trace, buffers = [], {}
    backend = S.CudaRefreshBackend(opt, wl.beta, wl.nesterov)
    plan = S.bucketed_refresh_step(shapes, P, Gd, Md, backend, bucket_bytes=40 << 20, buffers=buffers, trace=trace)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    assert len(plan[2]) >= 3 and trace[:3] == [("gather", 0), ("gather", 1), ("refresh", 0)]
    for i in range(len(shapes)):
        assert np.array_equal(U.to_np64(Md[i]), Mu[i])
        assert U.rel_fro(U.to_np64(P[i]), Wu[i]) <= 2e-2
    # a second call reuses the buffers
    keep = buffers["recv"][0].data_ptr()
    S.bucketed_refresh_step(shapes, P, Gd, Md, backend, bucket_bytes=40 << 20, buffers=buffers)
    assert buffers["recv"][0].data_ptr() == keep
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    opt.close()


@pytest.mark.gpu
def test_refresh_gathered_rejects_bad_arguments():
    shapes = [(64, 128)]
    opt = B.PeriodicRowwiseMuon(shapes, 1)
    buf = torch.zeros(64 * 128, dtype=torch.bfloat16, device="cuda")
    p = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    with pytest.raises(B.PrmError) as e:       # segment too small for the matrix
        B.prm_refresh_gathered(opt.h, [0], buf.data_ptr(), 64 * 128 - 8, [0], 1, 0, [p.data_ptr()], s)
    assert e.value.code == B.PRM_ERR_SHAPE
    with pytest.raises(B.PrmError) as e:
        B.prm_refresh_gathered(opt.h, [1], buf.data_ptr(), 64 * 128, [0], 1, 0, [p.data_ptr()], s)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_refresh_gathered(opt.h, [0], buf.data_ptr(), 64 * 128, [0], 2, 2, [p.data_ptr()], s)
    assert e.value.code == B.PRM_ERR_ARG
    with pytest.raises(B.PrmError) as e:
        B.prm_refresh_gathered(opt.h, [0], buf.data_ptr(), 64 * 128, [0], 1, 0, [0], s)
    assert e.value.code == B.PRM_ERR_ARG
    torch.cuda.synchronize()
    assert not p.any() and opt.status() == B.PRM_OK
    opt.close()


@pytest.mark.gpu
def test_bench_sharded_mode_single_rank_line():
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--sharded", "--config", "2", "--blocks", "2",
                        "--K", "2", "--steps", "4", "--warmup", "3", "--bucket-mib", "64"], env=env,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-800:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["scaling"] == "strong" and line["n_gpus"] == 1 and line["unit"] == "ms/step"
    assert line["refresh_ms"] > line["row_step_ms"] > 0
    pipe = line["pipeline"]
    assert pipe["buckets"] == line["config"]["buckets"] >= 3
    # the model's makespan lies between the compute alone and compute plus communication
    assert pipe["compute_ms_sum"] <= pipe["t_pipe_model_ms"] <= pipe["compute_ms_sum"] + pipe["gather_ms_sum"] + 1e-6
    assert pipe["gathered_payload_bytes"] == 2 * 2 * 18 * 2048 * 2048


def test_partition_matrices_is_balanced_and_deterministic():
    for cfg_id, world in ((4, 8), (2, 3), (3, 5), (5, 7)):
        shapes = [tuple(s) for s in workload(cfg_id).shapes]
        owner, load = B.prm_partition_matrices(shapes, world)
        assert len(owner) == len(shapes) and set(owner) == set(range(world))
        # the flop the default NS5 schedule executes: 8 r^2 c + 13 r^3 (c > 2r), 9 r^2 c + 11 r^3
        # (c >= 1.5 r), 15 r^2 c + 5 r^3 otherwise (all of these shapes have r >= 1024)
        def flop(s):
            r, c = min(s), max(s)
            k = (8, 13) if c > 2 * r else ((9, 11) if 2 * c >= 3 * r else (15, 5))
            return k[0] * r * r * c + k[1] * r ** 3
        cost = [flop(s) for s in shapes]
        for q in range(world):
            assert load[q] == pytest.approx(sum(c for c, o in zip(cost, owner) if o == q), rel=1e-12)
        # greedy longest-processing-time: no rank exceeds the mean by more than the largest matrix
        assert max(load) <= sum(cost) / world + max(cost)
        assert max(load) / (sum(cost) / world) < 1.1
        assert B.prm_partition_matrices(shapes, world)[0] == owner
    # brute force on a tiny case: the greedy result is within the list-scheduling bound of the optimum
    shapes = [(8, 8), (8, 16), (8, 24), (8, 8), (8, 32)]
    owner, load = B.prm_partition_matrices(shapes, 2)
    cost = [15 * 64 * c + 5 * 512 for (_, c) in shapes]
    best = min(max(sum(c for c, bit in zip(cost, range(5)) if (mask >> bit) & 1),
                   sum(c for c, bit in zip(cost, range(5)) if not (mask >> bit) & 1)) for mask in range(32))
    assert best <= max(load) <= (4 / 3 - 1 / 6) * best
    assert B.prm_partition_matrices([(4, 4)], 3)[0] == [0]
    with pytest.raises(B.PrmError):
        B.prm_partition_matrices([(4, 4)], 0)


def test_planning_functions_on_random_inputs():
    from hypothesis import given, settings, strategies as st

    shape = st.tuples(st.integers(1, 5000), st.integers(1, 5000))

    @settings(max_examples=150, deadline=None)
    @given(st.lists(shape, min_size=1, max_size=12), st.integers(1, 9), st.integers(1, 1 << 26))
    def plan(shapes, world, cap):
        want = O.bucket_plan(shapes, world, cap)
        got = B.prm_bucket_plan(shapes, world, cap)
        assert list(got[0]) == want[0] and list(got[1]) == want[1] and list(got[2]) == want[2]
        _check_plan(shapes, world, cap, got)

    @settings(max_examples=150, deadline=None)
    @given(st.integers(1, 1 << 20), st.integers(1, 64))
    def rows(n, world):
        covered = 0
        for q in range(world):
            lo, cnt = B.prm_shard_rows(n, world, q)
            assert (lo, cnt) == O.shard_rows(n, world, q)
            assert lo == min(n, covered) and cnt >= 0
            covered += cnt
        assert covered == n

    plan()
    rows()
