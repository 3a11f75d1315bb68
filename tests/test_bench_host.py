"""Host-side logic of bench.py: flop and byte accounting, and the N > 1 path
(independent replicas; the only cross-rank traffic is the max over ranks of
the timings), exercised with two gloo ranks on CPU."""

import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as td
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench
from paper_2608_20818_b200 import binding as B  # noqa: E402
from paper_2608_20818_b200.workloads import workload  # noqa: E402


def test_accounting_matches_the_shape_sets():
    # per block: 18 d^2 elements; executed flop 15 r^2 c + 5 r^3, model 20 r^2 c + 10 r^3
    for cfg, d, blocks in ((2, 2048, 24), (3, 3072, 36), (4, 4096, 42), (5, 5120, 48)):
        wl = workload(cfg)
        assert len(wl.shapes) == 5 * blocks
        assert bench.elements(wl.shapes) == 18 * d * d * blocks
        ex, mo = bench.ns5_flops(wl.shapes)
        assert mo == 410 * d ** 3 * blocks          # 70 + 30 + 90 + 90 + 130 per block
        assert ex == 295 * d ** 3 * blocks          # 50 + 20 + 65 + 65 + 95 per block
        # what the library reports with its default schedule (first three iterations in Gram space
        # for c >= 1.5 r, last Gram matrix by recurrence for c > 2 r): 8 r^2 c + 13 r^3
        h = B.prm_create([tuple(sh) for sh in wl.shapes], 5, 0.95, True, 1e-3, 0.0)
        n_groups = B.prm_plan(h, 0, len(wl.shapes))[1]
        info = [B.prm_group_info(h, g) for g in range(n_groups)]
        B.prm_destroy(h)
        flop = {(g["rows"], g["cols"]): g["ns5_flop"] for g in info}
        ex_lib, mo_lib = bench.ns5_flops(wl.shapes, flop)
        assert mo_lib == mo and ex_lib == 208 * d ** 3 * blocks     # 37 + 20 + 45 + 45 + 61 per block
    ex, mo = bench.ns5_flops(workload(4).shapes)
    assert abs(ex / 1e12 - 851.4) < 0.1 and abs(mo / 1e12 - 1183.3) < 0.1
    assert abs(14 * bench.elements(workload(4).shapes) / 1e9 - 177.6) < 0.1


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    td.init_process_group("gloo", rank=rank, world_size=world)
    got = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0])
    td.barrier()
    td.destroy_process_group()
    q.put((rank, got))


def test_max_over_ranks_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert out[0] == out[1] == [2.0, 10.0, 5.0]
    assert bench.per_replica_ms(100.0, 2) == 50.0
    assert bench.max_over_ranks([3.0]) == [3.0]          # not distributed: identity


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--config", "2"], env=env, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "ms/step" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["value"] > 0


def test_gpus_flag_launches_the_ranks_and_partitions_whole_matrices():
    """`bench.py --gpus 2` with no launcher around it starts two ranks itself
    (gloo on CPU in --dry-run).  Under --partition matrices every matrix of the
    set belongs to exactly one rank, and the printed line says n_gpus: 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR",
                                                            "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--partition", "matrices",
                        "--config", "2", "--dry-run"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-800:]
    lines = [json.loads(x) for x in r.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1, "rank 0 alone prints"
    line = lines[0]
    assert line["n_gpus"] == 2 and line["scaling"] == "strong" and line["partition"] == "matrices"
    lists = line["matrix_lists"]
    n = len(workload(2).shapes)
    assert len(lists) == 2
    assert sorted(lists[0] + lists[1]) == list(range(n)), "union is the whole set, no matrix twice"
    assert not set(lists[0]) & set(lists[1])
    cost = line["ns5_flop_per_rank"]
    assert max(cost) <= 1.1 * (sum(cost) / 2), "balanced within 10 % of the mean"
    # the same lists as the host planner gives directly
    owner, _ = B.prm_partition_matrices([tuple(s) for s in workload(2).shapes], 2)
    assert lists == [[i for i, q in enumerate(owner) if q == k] for k in range(2)]


def test_replicas_dry_run_and_world_size_mismatch():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--config", "2", "--dry-run"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-800:]
    line = [json.loads(x) for x in r.stdout.splitlines() if x.startswith("{")][0]
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert line["matrix_lists"][0] == line["matrix_lists"][1] == list(range(len(workload(2).shapes)))
    # a launcher that started another number of ranks than --gpus says is an error, not a silent n_gpus: 1
    env2 = dict(env, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env2,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "does not match" in r.stderr
