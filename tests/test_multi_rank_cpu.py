"""Host logic of the N > 1 path (independent replicas, no data-path collective), on CPU with gloo:
max-over-ranks timing, whole-job aggregation, and the reference arm's "rank 0 only" rule."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_info() == (world, rank, rank)
    ms = 10.0 + 5.0 * rank                        # rank 1 is the slow replica
    slowest = bench.max_over_ranks(ms, world)
    value = bench.aggregate_throughput(117.05, slowest / 1e3, world)
    dist.barrier()
    q.put((rank, slowest, value))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_summed_units():
    world, port = 2, 29533
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 15.0
        assert abs(value - 2 * 117.05 / 0.015) < 1e-6


def test_single_rank_helpers_need_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate_throughput(10.0, 2.0, 1) == 5.0
    wl = bench.inputs.WORKLOADS["c3_wan720p"]
    assert abs(bench.full_flops(wl) / 1e12 - 117.05) < 0.01
    import numpy as np
    assert abs(bench.computed_flops(wl, np.ones(256, np.uint8)) - bench.full_flops(wl)) < 1e3
    assert abs(bench.merge_bytes(wl, 4) / 1e9 - 25.8) < 0.1 and abs(bench.plan_bytes(wl) / 1e6 - 193.5) < 0.1


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", LOCAL_RANK="1", RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "c0_correctness", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = env["LOCAL_RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "c0_correctness", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
