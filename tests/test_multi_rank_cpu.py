"""Host logic of the N > 1 paths, on CPU with gloo: independent replicas (no data-path collective) with
max-over-ranks timing, whole-job aggregation and the reference arm's "rank 0 only" rule; and head sharding, whose
one exchange is the all-reduce of the plan's sums."""
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


def _shard_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import numpy as np
    from oracle import oracle as orc
    from paper_2607_15650_b200 import sharding
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, H, L, P = 2, 5, 97, 4
    off = orc.uniform_offsets(L, P)
    rng = np.random.default_rng(7)                       # the same LSE cache on every rank; each keeps its heads
    lse = rng.normal(0.0, 2.0, size=(P, B, H, L)) + np.linspace(0.0, 3.0, P)[:, None, None, None]
    h0, h1 = sharding.head_range(H, world, rank)
    n_i = np.diff(off).astype(np.float64)
    # this rank's sums of the per-row weights (Eq. 8): its mean times the rows it covers
    sums = orc.contribution(lse[:, :, h0:h1], off) * (B * (h1 - h0) * n_i)[:, None]
    t = torch.from_numpy(np.ascontiguousarray(sums).reshape(-1))
    sharding.all_reduce_sums(t)
    W = t.numpy().reshape(P, P) / (B * H * n_i)[:, None]
    W_all = orc.contribution(lse, off)
    mask, eps, K = orc.target_fraction(W, 0.5)
    mask_all, eps_all, K_all = orc.target_fraction(W_all, 0.5)
    q.put((rank, (h0, h1), float(np.abs(W - W_all).max()), bool((mask == mask_all).all()), abs(eps - eps_all),
           bool((orc.threshold(W, 0.2) == orc.threshold(W_all, 0.2)).all()), W.tobytes()))
    dist.barrier()
    dist.destroy_process_group()


def test_head_shards_reach_one_plan_through_an_all_reduce_of_sums():
    world, port = 2, 29537
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [(0, 3), (3, 5)]
    for rank, _, w_err, mask_same, eps_err, thr_same, _ in got:
        assert w_err < 1e-14 and mask_same and eps_err < 1e-14 and thr_same
    assert got[0][6] == got[1][6]                        # every rank holds the same totals, bit for bit


def test_head_range_covers_every_head_once():
    from paper_2607_15650_b200 import sharding
    import pytest
    for H, world in [(40, 8), (24, 8), (48, 5), (7, 7), (5, 2)]:
        spans = [sharding.head_range(H, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == H
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [b - a for a, b in spans]
        assert max(sizes) - min(sizes) <= 1 and sorted(sizes, reverse=True) == sizes
    with pytest.raises(ValueError):
        sharding.head_range(3, 4, 0)
    with pytest.raises(ValueError):
        sharding.head_range(8, 2, 2)
    t = torch.ones(4, dtype=torch.float64)
    assert sharding.all_reduce_sums(t) is t and float(t.sum()) == 4.0     # no process group: one shard
    with pytest.raises(TypeError):
        sharding.all_reduce_sums(torch.ones(4))


def test_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself (the same code path the GPU bench
    takes; here the ranks only join a gloo group and count themselves)."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--probe-world"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(x) for x in r.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1 and lines[0]["world_size"] == 2 and lines[0]["ranks_counted"] == 2 and lines[0]["n_gpus"] == 2
