#!/usr/bin/env python
"""Benchmark of the Periodic Row-wise Muon optimizer step on B200.

    python bench.py [--gpus N] [--steps S] [--warmup W] [--config 4] [--K 5]
    python bench.py --gpus N --partition matrices    # whole matrices dealt out to the N ranks
    python bench.py --impl reference ...      # the fp64 CPU oracle on the host cores

One "step" is one prm_step over the whole shape set (a refresh when
step_idx mod K == 0, a row step otherwise).  The line printed by rank 0 holds
the amortised optimizer ms/step at K, with per-branch times, the row-step
GB/s, the NS5 TFLOP/s, a roofline entry for the dominant kernel and the
oracle's CPU baseline.

With --gpus N > 1 and no launcher around it (WORLD_SIZE unset) the script
starts its own N ranks through torch.distributed.run on 127.0.0.1; under
torchrun it is one of the ranks.  N ranks are N independent replicas (weak
scaling, the default), or share one shape set: by whole matrices
(--partition matrices: no optimizer collective, NS5 work divided) or by rows
(--sharded: the paper's Algorithm 2, NS5 replicated).
"""

from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_20818_b200.workloads import (NS_WORKSPACE_BYTES_WHEN_FULL, RESERVE_BYTES, blocks_that_fit,  # noqa: E402
                                             make_grad, make_momentum, make_param, workload)

METRIC = "amortised optimizer ms/step at K"
NOMINAL_HBM_GBS = 8000.0       # nominal figure the targets are quoted against
NOMINAL_BF16_TFLOPS = 2250.0
GEMM_CLASSES = ("gram", "poly", "update", "update_final", "gramspace")
# DRAM traffic of the kernels, from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum) of a
# one-block case of the 9B-class set, scaled to a full launch by the work it processes (traffic
# grows in proportion to it).
GEMM_DRAM_BYTES_PER_EXEC_FLOP = 1449.7e6 / (8 * 4096 ** 2 * 12288 + 13 * 4096 ** 3)   # all 18 products of one matrix
ROW_DRAM_BYTES_PER_ELEMENT = {"wide": 14.0, "tall": 20.0,    # the tall matrices take two passes over g and m,
                              "tall_stream": 13.6}           # one with the streaming kernel


# ----------------------------------------------------------------- accounting
def ns5_flops(shapes, exec_flop=None):
    """(executed, paper model) flop of one refresh.  Executed: what the library
    reports per matrix of each shape (exec_flop: {shape: flop}, from
    prm_group_info: 9r^2c+11r^3 or 8r^2c+13r^3 where the first iterations run in
    Gram space), else the printed recurrence with triangle-only symmetric
    products, 15r^2c+5r^3."""
    ex = mo = 0
    for (m, n) in shapes:
        r, c = min(m, n), max(m, n)
        if exec_flop and (m, n) in exec_flop:
            ex += exec_flop[(m, n)]
        else:
            ex += 15 * r * r * c + 5 * r ** 3
        mo += 20 * r * r * c + 10 * r ** 3
    return ex, mo


def elements(shapes):
    return sum(m * n for (m, n) in shapes)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------ multi-GPU
def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default
    process group; the list itself when the job is not distributed.  The
    replicas exchange nothing else: timings are the only cross-rank traffic."""
    import torch.distributed as td
    if not (td.is_available() and td.is_initialized()) or td.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    td.all_reduce(t, op=td.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def per_replica_ms(job_ms, world):
    """N replicas advance N optimizer steps in job_ms: the whole-job figure is
    the time per replica-step."""
    return job_ms / world


# --------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "200"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                pw.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_median=statistics.median(pw), power_w_max=max(pw))
        return out


# ----------------------------------------------------------------- CPU oracle
def oracle_sample(wl, K, limit_s=20.0):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload
    and scales it to the whole shape set.  The sample is one matrix of each of
    the cheapest distinct shapes OF THE SET, as many as are predicted to fit the
    time limit and always at least the cheapest one (never a shape outside the
    set); each gets one refresh and one row step.  The refresh is scaled by the
    paper's flop model 20r^2c+10r^3, the row step by element count."""
    import numpy as np
    from oracle import prm_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    cfg = O.OracleConfig(K=K, beta=wl.beta, nesterov=wl.nesterov, lr=wl.lr, wd=wl.wd, gamma=wl.gamma)
    rng = np.random.default_rng(20818)

    def one(shape, t):
        W = rng.standard_normal(shape) * 0.02
        G = rng.standard_normal(shape) * wl.grad_std
        M = rng.standard_normal(shape) * wl.grad_std
        t0 = time.perf_counter()
        O.step_matrix(W, G, M, t, cfg)
        return time.perf_counter() - t0

    def model(shape):
        r, c = min(shape), max(shape)
        return 20.0 * r * r * c + 10.0 * r ** 3

    distinct = []
    for sh in wl.shapes:
        if sh not in distinct:
            distinct.append(sh)
    distinct.sort(key=model)
    # untimed probe (not part of the sample): the host's matmul rate, to predict what fits
    probe = (min(512, min(distinct[0])),) * 2
    one(probe, 0)
    rate = model(probe) / max(one(probe, 0), 1e-6)
    sample, predicted = [], 0.0
    for sh in distinct:
        if sample and predicted + model(sh) / rate > limit_s:
            break
        sample.append(sh)
        predicted += model(sh) / rate
    t_ref = sum(one(sh, 0) for sh in sample)
    t_row = sum(one(sh, 1) for sh in sample) if K > 1 else 0.0
    _, total_model = ns5_flops(wl.shapes)
    ref_ms = 1e3 * t_ref * total_model / sum(model(sh) for sh in sample)
    row_ms = 1e3 * t_row * elements(wl.shapes) / float(sum(m * n for (m, n) in sample))
    amort = (ref_ms + (K - 1) * row_ms) / K
    txt = (f"one refresh and one row step of the oracle on one matrix each of {sample} "
           f"({t_ref:.2f} s, {t_row:.3f} s), scaled to the shape set by the 20r^2c+10r^3 flop model "
           f"(refresh) and by element count (row step)")
    return {"value": amort, "unit": "ms/step", "cores": cores, "kind": "oracle", "sample": txt,
            "shapes_sampled": "%d of %d distinct shapes of the set" % (len(sample), len(distinct)),
            "refresh_ms": ref_ms, "row_step_ms": row_ms}


def run_reference(args, wl, K):
    """The reference arm: the oracle as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    base = None
    per = max(2.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        base = oracle_sample(wl, K, limit_s=per)
        if i >= args.warmup:
            vals.append(base["value"])
    v = sum(vals) / len(vals)
    base["value"] = v
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "ms/step", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "K": K, "matrices": len(wl.shapes)},
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": "ms/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------- GPU arm
def run_sharded(args, wl, K, rank, local_rank, world, dev):
    """Algorithm 2 over `world` ranks: every matrix is split by rows; refresh
    steps run the bucketed all-gather pipeline (every rank runs NS5 on every
    matrix, as in the paper), the other steps the sharded row step.  Strong
    scaling: the shape set is fixed, the rows per rank shrink with N.  Beside
    the step times it measures, bucket by bucket, the all-gather time a_l and
    the compute time c_l in isolation and evaluates the ideal two-stage
    pipeline model on them."""
    import math
    import torch.distributed as td
    from paper_2608_20818_b200 import binding as B
    from paper_2608_20818_b200 import sharded as S

    shapes = [tuple(s) for s in wl.shapes]
    n = len(shapes)
    dist = world > 1
    opt = B.PeriodicRowwiseMuon(shapes, K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma, io_dtype=wl.io_dtype,
                                gram_span=0 if args.printed_ns5 else args.ns5_schedule, device=dev)

    def shard(t, rows):
        lo, cnt = B.prm_shard_rows(rows, world, rank)
        return t[lo:lo + cnt].clone()

    params = [shard(make_param(wl, i, dev), shapes[i][0]) for i in range(n)]
    moms = [shard(make_momentum(wl, i, dev), shapes[i][0]) for i in range(n)]
    grads = [shard(make_grad(wl, i, 0, dev), shapes[i][0]) for i in range(n)]
    wide = [i for i in range(n) if shapes[i][0] <= shapes[i][1] and params[i].shape[0] > 0]
    tall = [(params[i], grads[i], moms[i], shapes[i][0]) for i in range(n)
            if shapes[i][0] > shapes[i][1] and params[i].shape[0] > 0]
    # rows of a wide matrix are local: their row step runs through a handle over the local shapes
    opt_wide = B.PeriodicRowwiseMuon([tuple(params[i].shape) for i in wide], K, wl.beta, wl.nesterov, wl.lr, wl.wd,
                                     gamma=wl.gamma, io_dtype=wl.io_dtype, no_refresh=True, ns_workspace_bytes=1,
                                     device=dev) if wide else None
    tall_backend = S.CudaTallBackend(wl.beta, wl.nesterov, wl.lr, wl.wd, wl.gamma, 1e-8)
    refresh_backend = S.CudaRefreshBackend(opt, wl.beta, wl.nesterov)
    buffers = {}
    stream = torch.cuda.current_stream(dev)
    cap = args.bucket_mib << 20

    def wide_step():
        if opt_wide is not None:
            opt_wide.step([params[i] for i in wide], [grads[i] for i in wide], [moms[i] for i in wide], 1)

    def step(t):
        if t % K == 0:
            S.bucketed_refresh_step(shapes, params, grads, moms, refresh_backend, bucket_bytes=cap, buffers=buffers,
                                    exchange=args.exchange)
        else:
            S.sharded_row_step(tall, wide_step, tall_backend, stream=stream.cuda_stream)

    def barrier():
        if dist:
            td.barrier()
        torch.cuda.synchronize()

    t = (K - (args.warmup % K)) % K
    for _ in range(args.warmup):
        step(t)
        t += 1
    barrier()
    assert opt.status() == B.PRM_OK
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    kinds = []
    barrier()
    ev[0].record(stream)
    for k in range(args.steps):
        kinds.append(t % K == 0)
        step(t)
        ev[k + 1].record(stream)
        t += 1
    barrier()
    clocks = sampler.stop() if sampler else None
    assert opt.status() == B.PRM_OK
    per_step = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    ref_ms = [x for x, r in zip(per_step, kinds) if r]
    row_ms = [x for x, r in zip(per_step, kinds) if not r]
    total_ms = ev[0].elapsed_time(ev[args.steps])

    # per-bucket times in isolation: gather alone, then rebuild + NS5 + slice alone
    bucket_of_mat, offsets, segments = B.prm_bucket_plan(shapes, world, cap)
    a_ms, c_ms = [], []
    if args.exchange == "p2p":          # no separate transfer to time: the rebuild does the reading
        buffers = {"send": buffers["send"],
                   "recv": [torch.empty(max(segments) * world, dtype=torch.bfloat16, device=dev)]}
    for l, seg in enumerate(segments):
        members = [i for i in range(n) if bucket_of_mat[i] == l]
        send = buffers["send"][0][:seg]
        recv = buffers["recv"][0][:seg * world]
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        barrier()
        e[0].record(stream)
        if dist:
            td.all_gather_into_tensor(recv, send)
        else:
            recv.copy_(send)
        e[1].record(stream)
        refresh_backend.refresh(members, recv, seg, [offsets[i] for i in members], world, rank,
                                [params[i] for i in members], stream.cuda_stream)
        e[2].record(stream)
        barrier()
        a_ms.append(e[0].elapsed_time(e[1]))
        c_ms.append(e[1].elapsed_time(e[2]))
    a_ms = max_over_ranks(a_ms, dev)
    c_ms = max_over_ranks(c_ms, dev)
    total_ms, mean_ref, mean_row = max_over_ranks(
        [total_ms, sum(ref_ms) / max(1, len(ref_ms)), sum(row_ms) / max(1, len(row_ms))], dev)
    if rank != 0:
        return
    t_pipe, t_exposed = B.prm_pipeline_model(a_ms, c_ms)
    amort = (mean_ref + (K - 1) * mean_row) / K if (ref_ms and (row_ms or K == 1)) else total_ms / args.steps
    out = {
        "metric": METRIC, "value": amort, "unit": "ms/step", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": False, "scaling": "strong", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "K": K, "matrices": n, "blocks": wl.blocks, "d": wl.d,
                   "parallelism": "rows sharded over %d ranks (Algorithm 2), NS5 replicated" % world,
                   "bucket_mib": args.bucket_mib, "buckets": len(segments), "exchange": args.exchange,
                   "l2": "inputs larger than L2"},
        "refresh_ms": mean_ref if ref_ms else None, "row_step_ms": mean_row if row_ms else None,
        "clocks": clocks,
        "pipeline": {"buckets": len(segments), "gather_ms_sum": sum(a_ms), "compute_ms_sum": sum(c_ms),
                     "t_pipe_model_ms": t_pipe, "t_comm_exposed_model_ms": t_exposed,
                     "gathered_payload_bytes": sum(segments) * 2 * world,
                     "note": "a_l and c_l timed bucket by bucket in isolation (max over ranks); the model is "
                             "Eq. app-pipeline-time; refresh_ms is the pipelined step, which also packs the momentum"},
    }
    print(json.dumps(out))


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="prm", choices=["prm", "reference"])
    ap.add_argument("--config", type=int, default=4, help="benchmark configuration 2..5 (default 4: 9B-class)")
    ap.add_argument("--blocks", type=int, default=None, help="override the number of transformer blocks")
    ap.add_argument("--K", type=int, default=None)
    ap.add_argument("--check-mode", action="store_true", help="NS5 in fp32 on CUDA cores")
    ap.add_argument("--first-step", type=int, default=None, help="step index of the first warm-up step")
    ap.add_argument("--printed-ns5", action="store_true",
                    help="all five NS5 iterations as printed (no Gram-space iterations); same as --ns5-schedule 0")
    ap.add_argument("--ns5-schedule", type=int, default=2, choices=[0, 1, 2],
                    help="PRM_OPT_NS_GRAM_SPAN: 0 printed recurrence, 1 first three iterations in Gram space, "
                         "2 (library default) also the last Gram matrix from the one before it")
    ap.add_argument("--tall-kernel", type=int, default=0, choices=[0, 1, 2],
                    help="PRM_OPT_TALL_KERNEL: 0/1 two passes over the tall matrices, 2 the single-pass streaming kernel")
    ap.add_argument("--wide-kernel", type=int, default=0, choices=[0, 1],
                    help="PRM_OPT_WIDE_KERNEL: 0 the persistent bulk-copy-fed row step of wide matrices, 1 one row per CTA")
    ap.add_argument("--ns-workspace-gib", type=float, default=None,
                    help="PRM_OPT_NS_WORKSPACE_BYTES in GiB (library default 8): matrices of a shape are refreshed in "
                         "sub-batches that fit")
    ap.add_argument("--split-input", action="store_true",
                    help="PRM_OPT_NS_SPLIT_INPUT: the NS5 input as two bf16 planes (accuracy option, + 4 r^2 c flop)")
    ap.add_argument("--partition", default="replicas", choices=["replicas", "matrices"],
                    help="N > 1: independent replicas (weak scaling), or one shape set whose matrices are dealt "
                         "out to the ranks by prm_partition_matrices (strong scaling, no optimizer collective)")
    ap.add_argument("--sharded", action="store_true",
                    help="the paper's distributed execution over the N ranks (rows sharded, bucketed all-gather "
                         "refresh, sharded tall RowNorm) instead of N independent replicas")
    ap.add_argument("--bucket-mib", type=int, default=240, help="--sharded: cap on one bucket's gathered payload")
    ap.add_argument("--exchange", default="allgather", choices=["allgather", "p2p"],
                    help="--sharded: NCCL all-gather per bucket, or no collective: the rebuild reads every rank's "
                         "segment in place through symmetric memory (peer loads over NVLink)")
    ap.add_argument("--no-printed", action="store_true", help="skip the extra refresh steps with the printed NS5")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run", action="store_true",
                    help="launcher and partition logic only, on CPU ranks (gloo): every rank plans its matrix list "
                         "and runs a stub step; no CUDA work, no timing claim")
    return ap.parse_args(argv)


def launch_ranks(n, argv):
    """Start n ranks of this script on this node through torch.distributed.run
    (rendezvous on 127.0.0.1) and pass their output through."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={n}",
           "--local-addr", "127.0.0.1", os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def rank_matrix_list(shapes, world, rank):
    """(indices into `shapes` owned by `rank`, NS5 cost per rank in flop) under
    the whole-matrix partition (prm_partition_matrices, a host-only call)."""
    from paper_2608_20818_b200 import binding as B
    owner, cost = B.prm_partition_matrices([tuple(s) for s in shapes], world)
    return [i for i, q in enumerate(owner) if q == rank], cost


def run_dry(args, wl, K, rank, world):
    """The N-rank plumbing without a GPU: each rank takes its matrix list, runs
    a stub step over it, and rank 0 gathers the lists and prints the line."""
    import torch.distributed as td
    dist = world > 1
    if dist:
        td.init_process_group("gloo")
    if args.partition == "matrices":
        mine, cost = rank_matrix_list(wl.shapes, world, rank)
    else:
        mine, cost = list(range(len(wl.shapes))), [float(ns5_flops(wl.shapes)[0])] * world
    t0 = time.perf_counter()
    touched = sum(wl.shapes[i][0] * wl.shapes[i][1] for i in mine)      # the stub step: walk the list
    stub_ms = (time.perf_counter() - t0) * 1e3
    (stub_ms,) = max_over_ranks([stub_ms])
    lists = [None] * world
    if dist:
        td.all_gather_object(lists, mine)
    else:
        lists = [mine]
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "partition": args.partition,
                          "scaling": "strong" if args.partition == "matrices" else "weak",
                          "config": {"workload": wl.name, "K": K, "matrices": len(wl.shapes)},
                          "matrix_lists": lists, "ns5_flop_per_rank": cost, "elements_rank0": touched,
                          "stub_ms": stub_ms}))
    if dist:
        td.barrier()
        td.destroy_process_group()


def main(argv=None):
    args = parse_args(argv)
    raw_argv = list(sys.argv[1:] if argv is None else argv)
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    launched = "WORLD_SIZE" in os.environ
    if args.gpus > 1 and not launched:
        # no launcher around this process: start the N ranks ourselves (the reference arm too:
        # its rank 0 prints, the others leave at once)
        raise SystemExit(launch_ranks(args.gpus, raw_argv))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={world}")

    full = workload(args.config)
    mem = None
    if args.impl == "prm" and not args.dry_run:
        torch.cuda.set_device(local_rank)
        free_b, total_b = torch.cuda.mem_get_info()
        mem = {"free_gib": round(free_b / 2 ** 30, 2), "total_gib": round(total_b / 2 ** 30, 2)}
        if args.blocks is None and full.blocks and args.partition == "replicas" and not args.sharded:
            # the largest block count of the configuration that this device holds (all of them on a
            # B200 for configurations 2-5 when its memory is free)
            args.blocks = blocks_that_fit(args.config, free_b)
            mem["blocks_that_fit"] = args.blocks
    wl = workload(args.config, args.blocks)
    K = args.K or wl.K
    if args.steps is None:
        args.steps = 2 * K
    if args.warmup is None:
        args.warmup = max(3, K)
    if args.impl == "reference":
        run_reference(args, wl, K)
        return
    if args.dry_run:
        run_dry(args, wl, K, rank, world)
        return

    from paper_2608_20818_b200 import binding as B

    dist = world > 1
    dev = torch.device("cuda", local_rank)
    if dist:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=dev)

    if args.sharded:
        run_sharded(args, wl, K, rank, local_rank, world, dev)
        if dist:
            td.destroy_process_group()
        return

    # ------------------------------------------------- this rank's matrices
    set_shapes = wl.shapes                       # the shape set the job as a whole steps
    part_cost = None
    if args.partition == "matrices" and world > 1:
        mine, part_cost = rank_matrix_list(wl.shapes, world, rank)
        wl = dataclasses.replace(wl, shapes=tuple(wl.shapes[i] for i in mine))
    n = len(wl.shapes)
    io_bytes = 4 if wl.io_dtype == "fp32" else 2
    resident = elements(wl.shapes) * (2 * io_bytes + 4)
    nearly_full = mem is not None and resident > 0.8 * mem["free_gib"] * 2 ** 30
    ns_cap = NS_WORKSPACE_BYTES_WHEN_FULL if nearly_full else None
    if args.ns_workspace_gib is not None:
        ns_cap = int(args.ns_workspace_gib * 2 ** 30)
    opt = B.PeriodicRowwiseMuon(wl.shapes, K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma,
                                io_dtype=wl.io_dtype, check_mode=args.check_mode,
                                gram_span=0 if args.printed_ns5 else args.ns5_schedule,
                                ns_workspace_bytes=ns_cap, tall_kernel=args.tall_kernel, split_input=args.split_input,
                                wide_kernel=args.wide_kernel, device=dev)
    gram_iters = {(g["rows"], g["cols"]): g["gram_iters"] for g in opt.groups()}
    exec_flop = {(g["rows"], g["cols"]): g["ns5_flop"] for g in opt.groups()}
    params = [make_param(wl, i, dev) for i in range(n)]
    moms = [make_momentum(wl, i, dev) for i in range(n)]
    # Gradients: every matrix owns its gradient buffer in HBM.  Two full sets (seeded for step 0 and
    # step 1) alternate from step to step where a second set fits beside the shape set; otherwise
    # one set is reused (timing does not depend on the values).
    free_now = torch.cuda.mem_get_info()[0]
    grad_bytes = elements(wl.shapes) * io_bytes
    n_sets = 2 if free_now - 2 * grad_bytes > RESERVE_BYTES else 1
    grad_sets = []
    for sset in range(n_sets):
        grad_sets.append([make_grad(wl, i, sset, dev) for i in range(n)])
    grads = grad_sets[0]
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream(dev)
    t_first = (K - (args.warmup % K)) % K            # so that the first timed step is a refresh
    if args.first_step is not None:
        t_first = args.first_step
    step_idx = t_first

    def barrier():
        if dist:
            td.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        opt.step(params, grad_sets[step_idx % n_sets], moms, step_idx)
        step_idx += 1
    barrier()
    assert opt.status() == B.PRM_OK, "device status after warm-up"

    launches0 = opt.launch_count()
    opt.profile(True)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    kinds = []
    barrier()
    ev[0].record(stream)
    for k in range(args.steps):
        kinds.append(opt.plan(step_idx)[0])
        opt.step(params, grad_sets[step_idx % n_sets], moms, step_idx)
        ev[k + 1].record(stream)
        step_idx += 1
    barrier()
    clocks = sampler.stop() if sampler else None
    prof = opt.profile_read()
    opt.profile(False)
    launches = opt.launch_count() - launches0
    assert opt.status() == B.PRM_OK, "device status after the timed region"

    per_step = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[args.steps])
    ref_ms = [t for t, r in zip(per_step, kinds) if r]
    row_ms = [t for t, r in zip(per_step, kinds) if not r]
    total_ms, mean_ref, mean_row = max_over_ranks(
        [total_ms, sum(ref_ms) / max(1, len(ref_ms)), sum(row_ms) / max(1, len(row_ms))], dev)

    # ---------------------------------------------------------- e2e (host grads)
    e2e = None
    if not args.no_e2e:
        # pinned host gradients: one matrix of each shape stands for every matrix of that shape
        by_shape = {}
        for i in range(n):
            if tuple(wl.shapes[i]) not in by_shape:
                hbuf = torch.empty(wl.shapes[i], dtype=grads[i].dtype).pin_memory()
                hbuf.copy_(grads[i])
                by_shape[tuple(wl.shapes[i])] = hbuf
        grads_host = [by_shape[tuple(wl.shapes[i])] for i in range(n)]
        readback = torch.empty(1024, dtype=params[0].dtype).pin_memory()
        h2d = sum(m * nn for (m, nn) in wl.shapes) * io_bytes
        d2h = readback.numel() * readback.element_size() + 4
        e_steps = args.steps
        barrier()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for k in range(e_steps):
            opt.step_h2d(params, grads, grads_host, moms, step_idx)
            readback.copy_(params[0].view(-1)[:1024], non_blocking=True)
            stream.synchronize()
            assert opt.status() == B.PRM_OK
            step_idx += 1
        t1.record(stream)
        barrier()
        (e_ms,) = max_over_ranks([t0.elapsed_time(t1) / e_steps], dev)
        weak = args.partition == "replicas"
        e2e = {"value": per_replica_ms(e_ms, world) if weak else e_ms, "unit": "ms/step", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h,
               "note": "gradients copied every step from pinned host memory (one matrix of each shape, reused "
                       "for every matrix of that shape) through prm_step_h2d; 2 KB of parameters and the status "
                       "word read back: this figure is the host link (PCIe), not the kernels"}

    # ------------------------------------------ the printed recurrence beside it
    # The same refresh with all five NS5 iterations evaluated as the paper prints them
    # (PRM_OPT_NS_GRAM_SPAN = 0), on the same buffers, so that the line carries both figures.
    printed = None
    if any(gram_iters.values()) and not args.check_mode and not args.no_printed:
        torch.cuda.empty_cache()
        opt0 = B.PeriodicRowwiseMuon(wl.shapes, K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma,
                                     io_dtype=wl.io_dtype, gram_span=0, ns_workspace_bytes=ns_cap, device=dev)
        p0 = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        barrier()
        for k in range(3):                       # one warm-up refresh, two timed
            if k == 1:
                opt0.profile(True)
            p0[k].record(stream)
            opt0.step(params, grads, moms, 0)
        p0[3].record(stream)
        barrier()
        prof0 = opt0.profile_read()
        assert opt0.status() == B.PRM_OK
        (ref0,) = max_over_ranks([p0[1].elapsed_time(p0[3]) / 2], dev)
        printed = {"refresh_ms": ref0,
                   "gemm_ms_per_refresh": sum(prof0[k][0] for k in GEMM_CLASSES) / 2}
        opt0.close()
        del opt0

    # --------------------------- the other tall-matrix row step beside it
    # Four row steps with the tall kernel that the main region did not use (two passes / single
    # pass), same buffers, so that one line carries both.
    tall_alt = None
    if any(sh[0] > sh[1] for sh in wl.shapes) and not args.no_printed and wl.io_dtype == "bf16":
        alt = 1 if args.tall_kernel == 2 else 2
        torch.cuda.empty_cache()
        opt1 = B.PeriodicRowwiseMuon(wl.shapes, K, wl.beta, wl.nesterov, wl.lr, wl.wd, gamma=wl.gamma,
                                     io_dtype=wl.io_dtype, ns_workspace_bytes=1, no_refresh=True, tall_kernel=alt,
                                     device=dev)
        barrier()
        for k in range(6):                       # two warm-up row steps, four timed
            if k == 2:
                opt1.profile(True)
            opt1.step(params, grads, moms, 1)
        barrier()
        prof1 = opt1.profile_read()
        assert opt1.status() == B.PRM_OK
        (alt_ms,) = max_over_ranks([prof1["row_tall"][0] / 4], dev)
        tall_alt = {"kernel": "single pass (streaming)" if alt == 2 else "two passes", "tall_ms_per_step": alt_ms,
                    "launches_per_step": prof1["row_tall"][1] // 4,
                    "note": "four row steps back to back after the main region (no refresh in between: SM clock "
                            "higher than inside the K-step period)"}
        opt1.close()
        del opt1

    if rank != 0:
        if dist:
            td.destroy_process_group()
        return

    pk = peaks()
    weak = args.partition == "replicas"
    amort = (mean_ref + (K - 1) * mean_row) / K if (ref_ms and (row_ms or K == 1)) else total_ms / args.steps
    n_ref, n_row = len(ref_ms), len(row_ms)
    ex, mo = ns5_flops(wl.shapes, exec_flop)
    ex_printed, _ = ns5_flops(wl.shapes)
    el = elements(wl.shapes)
    el_tall = elements([sh for sh in wl.shapes if sh[0] > sh[1]])
    row_bytes = el * (3 * io_bytes + 8)   # g and p read, p write (I/O dtype), m read and write (fp32)
    gemm_ms = sum(prof[k][0] for k in GEMM_CLASSES)
    gemm_launches = sum(prof[k][1] for k in GEMM_CLASSES)
    row_kernel_ms = prof["row_wide"][0] + prof["row_tall"][0]
    if world == 1:
        parallelism = "one GPU"
    elif weak:
        parallelism = "%d independent replicas" % world
    else:
        parallelism = "whole matrices dealt out to %d ranks (prm_partition_matrices), no optimizer collective" % world
    out = {
        "metric": METRIC, "value": per_replica_ms(amort, world) if weak else amort, "unit": "ms/step", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": False,
        "scaling": "weak" if weak else "strong", "vs_baseline": None,
        "dtype": "f32" if args.check_mode else "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "K": K, "matrices": len(set_shapes), "blocks": wl.blocks,
                   "blocks_stated": full.blocks, "d": wl.d,
                   "elements": elements(set_shapes), "io_dtype": wl.io_dtype, "momentum_dtype": "fp32",
                   "ns5": "fp32 check mode" if args.check_mode else "bf16 tcgen05",
                   "ns5_schedule": ("five iterations as printed" if not any(gram_iters.values()) else
                                    "PRM_OPT_NS_GRAM_SPAN=%d: iterations 1-3 in Gram space for %d of %d matrices%s" % (
                                        args.ns5_schedule, sum(1 for sh in wl.shapes if gram_iters.get(tuple(sh), 0)), n,
                                        ", last Gram matrix from the previous one where c > 2r"
                                        if args.ns5_schedule == 2 else "")),
                   "parallelism": parallelism, "matrices_rank0": n,
                   "device_memory": mem, "ns_workspace_cap_bytes": ns_cap,
                   "gradient_sets": n_sets,
                   "tall_row_step": "single pass (streaming)" if args.tall_kernel == 2 else "two passes",
                   "wide_row_step": "one row per CTA" if args.wide_kernel == 1 else "persistent, bulk copies",
                   "ns5_input": "two bf16 planes (PRM_OPT_NS_SPLIT_INPUT)" if args.split_input else "bf16",
                   "l2": "inputs larger than L2 (working set %.1f GB)" % (el * 8 / 1e9),
                   "first_timed_step_index": t_first + args.warmup},
        "refresh_ms": mean_ref if n_ref else None, "row_step_ms": mean_row if n_row else None,
        "refresh_steps_timed": n_ref, "row_steps_timed": n_row,
        "per_step_ms": [round(t, 3) for t in per_step],       # rank 0, in order; refresh steps are the large ones
        "gpu_launches": launches,
        "clocks": clocks,
        # device time per kernel class over the whole timed region (CUDA events inside the library)
        "kernel_classes": {k: {"ms": round(v[0], 3), "launches": v[1]} for k, v in prof.items()},
    }
    if part_cost is not None:
        out["config"]["ns5_flop_per_rank"] = part_cost
    if n_row:
        gbs = row_bytes / (mean_row * 1e-3) / 1e9
        out["row_step"] = {"GB/s": gbs, "bytes_per_element": 3 * io_bytes + 8,
                           "frac_of_measured_peak": gbs / pk["hbm_gbs"], "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
                           "kernel_ms_per_step": row_kernel_ms / n_row,
                           "wide_ms_per_step": prof["row_wide"][0] / n_row, "tall_ms_per_step": prof["row_tall"][0] / n_row,
                           "tall_GB/s": (el_tall * (3 * io_bytes + 8) / (prof["row_tall"][0] / n_row * 1e-3) / 1e9
                                         if prof["row_tall"][0] > 0 else None)}
        if tall_alt is not None:
            tall_alt["tall_GB/s"] = el_tall * (3 * io_bytes + 8) / (tall_alt["tall_ms_per_step"] * 1e-3) / 1e9
            out["row_step"]["other_tall_kernel"] = tall_alt
    if n_ref and gemm_ms > 0:
        tf_exec = ex * n_ref / (gemm_ms * 1e-3) / 1e12
        out["ns5"] = {"TFLOP/s_exec": tf_exec,
                      "exec_flop_per_refresh": ex, "printed_flop_per_refresh": ex_printed,
                      "TFLOP/s_exec_whole_refresh": ex / (mean_ref * 1e-3) / 1e12,
                      "frac_of_measured_burst": tf_exec / pk["bf16_tflops"],
                      "frac_of_measured_sustained": tf_exec / pk["bf16_tflops_sustained"],
                      "frac_of_nominal_2250": tf_exec / NOMINAL_BF16_TFLOPS,
                      "gemm_ms_per_refresh": gemm_ms / n_ref, "prepass_ms_per_refresh": prof["prepass"][0] / n_ref,
                      # flop counts the kernels do NOT execute, over the same time: for comparison with the
                      # paper's accounting only
                      "model_equivalents": {"not_a_rate": True,
                                            "paper_model_20r2c_10r3": mo * n_ref / (gemm_ms * 1e-3) / 1e12,
                                            "printed_recurrence_symmetric": ex_printed * n_ref / (gemm_ms * 1e-3) / 1e12}}
        if args.check_mode:
            # fp32 FMA path: bounded by CUDA-core arithmetic, not by tensor cores
            peak = 148 * 128 * 2 * 1.965e9 / 1e12
            out["roofline"] = {"bound": "alu", "achieved": tf_exec, "peak": peak, "unit": "TFLOP/s",
                               "frac": tf_exec / peak, "traffic": None, "kernel": "gemm_simt_kernel",
                               "peak_source": "148 SMs x 128 fp32 FMA lanes x 2 flop x 1.965 GHz"}
        else:
            peak = pk["bf16_tflops_sustained"]
            out["roofline"] = {"bound": "tensor", "achieved": tf_exec, "peak": peak, "unit": "TFLOP/s",
                               "frac": tf_exec / peak,
                               "traffic": GEMM_DRAM_BYTES_PER_EXEC_FLOP * ex * n_ref / max(1, gemm_launches),
                               "traffic_unit": "DRAM bytes per launch, scaled from a one-block ncu capture",
                               "kernel": "gemm_tc_kernel",
                               "launches": gemm_launches, "avg_launch_ms": gemm_ms / max(1, gemm_launches),
                               "peak_source": "%s sustained bf16 matmul" % pk["source"]}
    elif n_row:
        gbs = row_bytes / (row_kernel_ms / n_row * 1e-3) / 1e9
        tall_key = "tall_stream" if args.tall_kernel == 2 else "tall"
        traffic = (ROW_DRAM_BYTES_PER_ELEMENT["wide"] * (el - el_tall) + ROW_DRAM_BYTES_PER_ELEMENT[tall_key] * el_tall)
        out["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                           "frac": gbs / pk["hbm_gbs"], "traffic": traffic,
                           "traffic_unit": "DRAM bytes per row step", "kernel": "rowstep_*",
                           "peak_source": "%s copy bandwidth" % pk["source"]}
    if printed is not None and n_ref:
        ex0, _ = ns5_flops(wl.shapes)
        v0 = (printed["refresh_ms"] + (K - 1) * mean_row) / K if (row_ms or K == 1) else printed["refresh_ms"]
        printed["value"] = per_replica_ms(v0, world) if weak else v0
        printed["TFLOP/s_exec_whole_refresh"] = ex0 / (printed["refresh_ms"] * 1e-3) / 1e12
        if printed["gemm_ms_per_refresh"] > 0:
            printed["TFLOP/s_exec"] = ex0 / (printed["gemm_ms_per_refresh"] * 1e-3) / 1e12
            if "roofline" in out and out["roofline"]["bound"] == "tensor":
                # the same kernel running the recurrence exactly as printed, against the same peak
                out["roofline"]["frac_printed_schedule"] = printed["TFLOP/s_exec"] / out["roofline"]["peak"]
        printed["note"] = ("all five NS5 iterations as printed (PRM_OPT_NS_GRAM_SPAN = 0), two refresh steps timed "
                           "after the main region; value = amortised ms/step with this refresh and the row step above")
        out["printed_ns5"] = printed
    out["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = oracle_sample(wl, K)
    print(json.dumps(out))
    if dist:
        td.destroy_process_group()


if __name__ == "__main__":
    main()
