#!/usr/bin/env python
"""Benchmark of the selective attention-state path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One timed "step" is one selective denoising step of the whole hot path on one attention layer:
dt_attn_states (COMPUTE pairs of the current plan) + dt_state_merge (all P states per row) +
dt_plan (contribution measure of the refreshed cache -> plan of the next step).  Before the timed
region an anchor step computes every pair and the first plan is derived from it.  Inputs (bf16
Q, K, V of every denoising step of the workload) are resident in HBM; they and the state cache
are far larger than L2, so no explicit flush is needed.

With N > 1 ranks each runs an independent replica of the layer (no collective); `--shard-heads` instead
spreads the heads of one layer over the ranks, with one all-reduce of the plan's P x S sums per step.

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead, on a
bounded sample of the same workload.
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

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_15650_b200 import inputs  # noqa: E402

# --policy alg1: (eps_local, cache ratio R) per workload, chosen so that the online policy computes about the share of
# pairs the fixed-fraction plans of the workload compute
ALG1_DEFAULTS = {"c3_wan720p": (0.0075, 0.85)}
METRIC = "effective_attn_tflops"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c3_wan720p"


# ------------------------------------------------------------------------------------------ helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.idx)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as fh:
            for line in fh:
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


def ncu_attn_traffic(workload: str):
    """DRAM bytes (read + written) of one attn_states_kernel launch per (head, COMPUTE pair), from the ncu capture
    that profiles/attn_states_traffic.json names (a capture on a few heads of the workload; the traffic grows in
    proportion to heads x pairs because the pair states written dominate it).  None if there is no capture."""
    path = os.path.join(ROOT, "profiles", "attn_states_traffic.json")
    if not os.path.exists(path):
        return None, None
    with open(path) as fh:
        rec = json.load(fh).get(workload)
    if not rec:
        return None, None
    per = (rec["dram_bytes_read"] + rec["dram_bytes_written"]) / (rec["heads"] * rec["computed_pairs"])
    return per, rec["capture"]


def full_flops(wl) -> float:
    return 4.0 * wl.L * wl.L * wl.D * wl.H * wl.B


def computed_flops(wl, mask: np.ndarray) -> float:
    n = np.diff(wl.offsets()).astype(np.float64)
    return 4.0 * wl.D * wl.H * wl.B * float((np.outer(n, n) * (mask.reshape(wl.P, wl.P) != 0)).sum())


def merge_bytes(wl, state_bytes: int, slots=None) -> float:
    S = wl.P if slots is None else slots
    return float(wl.L) * wl.H * wl.B * (S * (wl.D * state_bytes + 4) + 2 * wl.D + 4)


def plan_bytes(wl, slots=None) -> float:
    return float(wl.L) * wl.H * wl.B * (wl.P if slots is None else slots) * 4


def slot_members(P: int, g: int):
    """KV partitions behind every (query partition, slot) of a grouped cache: slot 0 = the local partition,
    slot 1 + k = group k of g adjacent partitions without the local one (structure only, no arithmetic)."""
    m = (P + g - 1) // g
    return [[[i]] + [[j for j in range(k * g, min(P, (k + 1) * g)) if j != i] for k in range(m)] for i in range(P)]


def slot_mask_to_pairs(mask: np.ndarray, P: int, g: int) -> np.ndarray:
    """[P][S] slot decisions -> the [P][P] pair mask they stand for."""
    if g <= 1:
        return mask.reshape(P, P)
    mem = slot_members(P, g)
    S = len(mem[0])
    mask = mask.reshape(P, S)
    pairs = np.zeros((P, P), np.uint8)
    for i in range(P):
        for sl in range(S):
            if mask[i, sl]:
                pairs[i, mem[i][sl]] = 1
    return pairs


def dist_info():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_ranks(n: int, argv, script=None) -> int:
    """`--gpus N` without a launcher around it: start N ranks of this script (one per GPU) under torch's launcher on
    127.0.0.1 and return its exit code.  With WORLD_SIZE already in the environment the caller is a rank and runs
    the bench itself instead."""
    script = script or os.path.abspath(__file__)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), script] + list(argv)
    return subprocess.run(cmd).returncode


def probe_world(args):
    """What a rank of `--gpus N --probe-world` does: join a gloo group on the CPU and let rank 0 print the world size
    (the launch path of the multi-GPU bench without a GPU)."""
    import torch.distributed as dist
    world, rank, local = dist_info()
    dist.init_process_group("gloo")
    t = torch.ones(1, dtype=torch.float64)
    dist.all_reduce(t)
    if rank == 0:
        print(json.dumps({"probe": "world", "world_size": dist.get_world_size(), "ranks_counted": int(t.item()),
                          "n_gpus": args.gpus}))
    dist.barrier()
    dist.destroy_process_group()


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Max of a per-rank scalar (the multi-rank timing rule); identity for one rank."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds_max: float, world: int) -> float:
    """Whole-job throughput of `world` independent replicas: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / seconds_max


# ------------------------------------------------------------------------------------------ oracle legs
def oracle_sample(wl, q, k, v, mask, budget_s: float, seed: int = 0, fp16: bool = False):
    """Time the oracle, as it stands, on a bounded sample: one head, a seeded subset of query rows;
    per row the COMPUTE pair states of its partition (Eq. 1) and the P-way merge (Eq. 2) -- REUSE
    states are taken as already cached (zeros stand in; the arithmetic cost is the same).
    Returns effective TFLOP/s (full-attention flops of the sampled rows / time), seconds, description."""
    from oracle import oracle as orc
    off = wl.offsets()
    rng = np.random.default_rng(seed)
    mask = mask.reshape(wl.P, wl.P)
    qb, kb, vb = (inputs.bf16_bits(x[:, :, :1].contiguous()) for x in (q, k, v))   # head 0 only

    def run(rows):
        t0 = time.perf_counter()
        part = np.searchsorted(off, rows, side="right") - 1
        o_st = np.zeros((rows.size, wl.P, wl.D)); l_st = np.full((rows.size, wl.P), -30.0)
        for i in range(wl.P):
            sel = np.nonzero(part == i)[0]
            if sel.size == 0:
                continue
            for j in range(wl.P):
                if mask[i, j]:
                    o, l = orc.pair_state(qb, kb, vb, wl.scale, 0, 0, rows[sel], int(off[j]), int(off[j + 1]), fp16=fp16)
                    o_st[sel, j], l_st[sel, j] = o, l
        orc.merge(o_st, l_st)
        return time.perf_counter() - t0

    n, t = min(256, wl.L), 0.0
    while True:                                   # grow the sample until it costs about budget_s
        rows = np.sort(rng.choice(wl.L, size=n, replace=False)).astype(np.int32)
        t = run(rows)
        if t >= 0.5 * budget_s or n == wl.L:
            break
        n = int(min(wl.L, max(2 * n, 0.9 * budget_s / max(t / n, 1e-9))))
    eff = 4.0 * n * wl.L * wl.D / t / 1e12
    desc = (f"fp64 oracle, head 0 of {wl.H}, {n} of {wl.L} query rows (seeded), COMPUTE pairs of the plan "
            f"({int(mask.sum())}/{wl.P * wl.P}) + {wl.P}-way merge; value = 4*rows*L*D/time")
    return eff, t, desc, orc.num_threads()


def run_reference(args, wl):
    world, rank, _ = dist_info()
    if rank != 0:
        return
    gen = inputs.StepInputs(wl, seed=0, device="cpu")
    q, k, v = gen.next()
    f = wl.fractions[-1]
    K = min(max(int(np.floor(f * wl.P * wl.P + 0.5)), wl.P), wl.P * wl.P)
    # banded plan with the target pair count (the oracle leg needs no GPU-derived plan)
    d = np.abs(np.subtract.outer(np.arange(wl.P), np.arange(wl.P)))
    order = np.argsort(d.reshape(-1), kind="stable")
    mask = np.zeros(wl.P * wl.P, np.uint8); mask[order[:K]] = 1
    budget = 5.0
    vals, secs = [], []
    for s in range(args.warmup + args.steps):
        eff, t, desc, cores = oracle_sample(wl, q, k, v, mask, budget, seed=s)
        if s >= args.warmup:
            vals.append(eff); secs.append(t)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "D": wl.D, "L": wl.L, "P": wl.P,
                   "computed_pair_fraction": K / (wl.P * wl.P)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ CUDA arm
def run_cuda(args, wl):
    from paper_2607_15650_b200 import binding, build, sharding
    world, rank, local = dist_info()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl_total = wl
    if args.shard_heads:     # one layer over all ranks: this rank keeps a contiguous share of the heads
        h0, h1 = sharding.head_range(wl.H, world, rank)
        wl = dataclasses.replace(wl, H=h1 - h0)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = load_peaks()
    state_dtype = binding.DT_STATE_BF16 if args.state_dtype == "bf16" else binding.DT_STATE_FP32
    sbytes = 2 if args.state_dtype == "bf16" else 4

    in_dt = torch.float16 if args.dtype == "fp16" else torch.bfloat16
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale, state_dtype, local, group_size=args.group_size,
                          input_dtype=binding.DT_INPUT_FP16 if args.dtype == "fp16" else binding.DT_INPUT_BF16)
    S, g = ctx.dt_num_slots()
    gen = inputs.StepInputs(wl, seed=rank if args.shard_heads else 0, device=dev, dtype=in_dt)
    steps_in = [gen.next() for _ in range(wl.steps)]          # resident bf16 inputs of every denoising step
    del gen
    torch.cuda.empty_cache()
    out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=in_dt, device=dev)
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    PP = wl.P * S            # decisions per plan: [P][S] (S = P without grouping)
    masks = [torch.ones(PP, dtype=torch.uint8, device=dev), torch.ones(PP, dtype=torch.uint8, device=dev)]
    ones = torch.ones(PP, dtype=torch.uint8, device=dev)
    W = torch.empty(PP, dtype=torch.float64, device=dev)
    sums = torch.empty(PP, dtype=torch.float64, device=dev)
    frac = args.fraction if args.fraction is not None else wl.fractions[-1]
    stream = torch.cuda.current_stream()

    if args.policy == "alg1":
        if world > 1 or args.group_size != 1:
            raise SystemExit("--policy alg1 is measured on one GPU with the pair cache")
        dflt = ALG1_DEFAULTS.get(wl.name, (0.01, 0.8))
        eps_local = args.eps_local if args.eps_local is not None else dflt[0]
        ratio = args.cache_ratio if args.cache_ratio is not None else dflt[1]
        n = max(args.steps, 2)
        measure_alg1(binding, dev, wl, ctx, steps_in, max(args.warmup, n // 2), eps_local, ratio, host_replay=False)
        rec = measure_alg1(binding, dev, wl, ctx, steps_in, n, eps_local, ratio, host_replay=not args.no_e2e)
        line = {"metric": METRIC, "value": rec["effective_tflops"], "unit": UNIT, "n_gpus": 1, "steps": n,
                "warmup": max(args.warmup, n // 2), "ms_per_step": rec["step_ms_mean"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
                "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "D": wl.D, "L": wl.L, "P": wl.P,
                           "policy": "alg1", "state_dtype": args.state_dtype,
                           "step": "dt_attn_local + dt_planner_step + dt_attn_states + dt_state_merge + dt_planner_commit",
                           "l2": "inputs and state cache larger than L2; no flush"},
                "clocks": rec["clocks"],
                "e2e": ({"value": full_flops(wl) / 1e12 / (rec["e2e_step_ms_mean"] / 1e3), "unit": UNIT,
                         "ms_per_step": rec["e2e_step_ms_mean"], "h2d_bytes_per_step": 3 * wl.B * wl.L * wl.H * wl.D * 2 + wl.P * wl.P,
                         "d2h_bytes_per_step": wl.B * wl.L * wl.H * (wl.D * 2 + 4), "includes": rec["e2e_includes"]}
                        if "e2e_step_ms_mean" in rec else None),
                "gpu_launches": None, "alg1": rec}
        print(json.dumps(line))
        return

    def plan(mask_buf):
        if args.shard_heads:   # local sums -> all-reduce of P*S doubles -> the same plan on every rank
            sharding.plan_sharded(ctx, wl_total.B * wl_total.H, mask_buf, sums, target_fraction=frac, w_dev=W)
        else:
            ctx.dt_plan(mask_buf, target_fraction=frac, w_dev=W)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def one_step(t, cur, timers=None):
        """dt_attn_states with plan `cur` -> dt_state_merge -> dt_plan into the other mask buffer."""
        q, k, v = steps_in[1 + (t % (wl.steps - 1))] if wl.steps > 1 else steps_in[0]
        if timers is not None:
            e = [ev() for _ in range(4)]
            e[0].record(stream)
        if args.fused:       # one pass: COMPUTE slots + composed reuse state -> output; no cache round trip, no re-plan
            ctx.dt_attn_fused(q, k, v, masks[cur], comp_o, comp_l, out, lse)
            if timers is not None:
                for i in (1, 2, 3):
                    e[i].record(stream)
                timers.append(e)
            return cur
        ctx.dt_attn_states(q, k, v, masks[cur], t)
        if timers is not None:
            e[1].record(stream)
        if args.composed:
            ctx.dt_state_merge_planned(masks[cur], comp_o, comp_l, out, lse)
        else:
            ctx.dt_state_merge(out, lse)
        if timers is not None:
            e[2].record(stream)
        plan(masks[cur ^ 1])
        if timers is not None:
            e[3].record(stream)
            timers.append(e)
        return cur if args.composed else cur ^ 1   # composed mode: the anchor's plan holds until the next anchor

    # anchor step: every pair computed, first plan derived from it
    q, k, v = steps_in[0]
    ctx.dt_attn_states(q, k, v, ones, 0)
    ctx.dt_state_merge(out, lse)
    plan(masks[0])
    comp_o = comp_l = None
    compose_ms = None
    if args.composed or args.fused:
        comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=ctx.o_state.dtype, device=dev)
        comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
        c0, c1 = ev(), ev()
        c0.record(stream)
        ctx.dt_compose_reuse(masks[0], comp_o, comp_l)
        c1.record(stream)
        torch.cuda.synchronize()
        compose_ms = c0.elapsed_time(c1)
    torch.cuda.synchronize()
    ctx.dt_poll()
    cur = 0
    t = 1
    for _ in range(args.warmup):
        cur = one_step(t, cur); t += 1
    torch.cuda.synchronize()

    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.dt_launch_count()
    timers = []
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for _ in range(args.steps):
        cur = one_step(t, cur, timers); t += 1
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    launches = ctx.dt_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ctx.dt_poll()
    total_ms = e0.elapsed_time(e1)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    attn_ms = [e[0].elapsed_time(e[1]) for e in timers]
    merge_ms = [e[1].elapsed_time(e[2]) for e in timers]
    plan_ms = [e[2].elapsed_time(e[3]) for e in timers]
    mask_np = slot_mask_to_pairs(masks[cur].cpu().numpy(), wl.P, g)   # as pairs: a slot stands for its members
    comp_fl = computed_flops(wl, mask_np)           # pair count is fixed by the target fraction
    n_comp = int((mask_np != 0).sum())
    n_slots_comp = int((masks[cur] != 0).sum().item())
    def job_throughput(seconds):   # whole job: N replicas of the layer, or one layer whose heads the ranks share
        if args.shard_heads:
            return full_flops(wl_total) / 1e12 / seconds
        return aggregate_throughput(full_flops(wl) / 1e12, seconds, world)

    value = job_throughput(ms_per_step / 1e3)

    # ---- end to end through the C ABI with host buffers (pinned): H2D of q, k, v, mask; D2H of out, lse
    e2e = None
    if not args.no_e2e:
        cfg = ctx.cfg
        ws = torch.empty(binding.dt_step_host_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
        qh, kh, vh = (x.cpu().pin_memory() for x in steps_in[1 % wl.steps])
        oh = torch.empty(out.shape, dtype=in_dt).pin_memory()
        lh = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        mh = masks[cur].cpu()
        times = []
        for i in range(1 + 3):
            if world > 1:
                import torch.distributed as dist
                dist.barrier()           # every replica runs its end-to-end step at the same time
            t0 = time.perf_counter()
            ctx.dt_step_host(qh, kh, vh, mh, t, oh, lh, ws)     # returns when out and lse are in host memory
            if not args.shard_heads:
                ctx.dt_plan(masks[cur ^ 1], target_fraction=frac, w_dev=W)   # the next step's plan, as in the timed loop
                torch.cuda.synchronize()
            times.append(time.perf_counter() - t0)
            t += 1
        e2e_s = max_over_ranks(float(np.mean(times[1:])), world, dev)
        h2d = 3 * qh.numel() * 2 + PP
        d2h = oh.numel() * 2 + lh.numel() * 4
        e2e = {"value": job_throughput(e2e_s), "unit": UNIT, "ms_per_step": 1e3 * e2e_s,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "includes": "dt_step_host: H2D q,k,v,mask + dt_attn_states + dt_state_merge + D2H out,lse; then dt_plan"}
        del ws

    if rank != 0:
        return

    # ---- all-compute plan on the same kernel (context for "ms/step vs full attention")
    full_ms = []
    for i in range(3 + 1):
        a, b, c = ev(), ev(), ev()
        q, k, v = steps_in[i % wl.steps]
        a.record(stream)
        ctx.dt_attn_states(q, k, v, ones, t)
        b.record(stream)
        ctx.dt_state_merge(out, lse)
        c.record(stream)
        torch.cuda.synchronize()
        t += 1
        if i > 0:
            full_ms.append((a.elapsed_time(b), b.elapsed_time(c)))
    full_attn_ms = float(np.mean([x[0] for x in full_ms]))
    full_step_ms = float(np.mean([x[0] + x[1] for x in full_ms]))
    dense_ms = []
    for i in range(3 + 1):          # plain full attention: every slot in one pass, nothing cached, nothing merged
        a, b = ev(), ev()
        q, k, v = steps_in[i % wl.steps]
        a.record(stream)
        ctx.dt_attn_fused(q, k, v, ones, None, None, out, lse)
        b.record(stream)
        torch.cuda.synchronize()
        if i > 0:
            dense_ms.append(a.elapsed_time(b))
    dense_ms = float(np.mean(dense_ms))

    # ---- CPU oracle on a bounded sample of the same workload
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        eff, secs, desc, cores = oracle_sample(wl, *steps_in[1 % wl.steps], mask_np, budget_s=15.0, fp16=args.dtype == "fp16")
        cpu = {"value": eff, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "seconds": secs}

    attn_avg_ms = float(np.mean(attn_ms))
    traffic_per, traffic_src = ncu_attn_traffic(args.workload)
    achieved = comp_fl / 1e12 / (attn_avg_ms / 1e3)
    peak = peaks["bf16_tflops_sustained"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if args.shard_heads else "weak",
        "vs_baseline": None,
        "dtype": args.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "H": wl_total.H, "heads_per_rank": wl.H, "D": wl.D, "L": wl.L, "P": wl.P,
                   "computed_pairs": n_comp, "computed_pair_fraction": n_comp / (wl.P * wl.P),
                   "group_size": g, "cache_slots": S, "computed_slots": n_slots_comp, "state_dtype": args.state_dtype,
                   "cache_gb": S * wl.B * wl.H * wl.L * (wl.D * sbytes + 4) / 1e9,
                   "step": ("dt_attn_fused (COMPUTE slots in one pass + composed reuse state in the epilogue)" if args.fused
                            else "dt_attn_states + dt_state_merge_planned + dt_plan" if args.composed
                            else "dt_attn_states + dt_state_merge + dt_plan"), "multi_gpu": ("heads sharded over the ranks; one all-reduce of P*S plan sums per step" if args.shard_heads
                                  else "independent replicas"),
                   "l2": "inputs (%.1f GB) and state cache larger than L2; no flush" %
                         ((3 * wl.L * wl.H * wl.D * 2) / 1e9)},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches,
        "roofline": {"kernel": "attn_states_kernel", "bound": "tensor", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak,
                     "traffic": (traffic_per * wl.H * n_comp
                                 if traffic_per is not None and args.state_dtype == "fp32" and g == 1 and args.dtype == "bf16"
                                 else None),
                     "traffic_note": f"bytes per launch: ncu dram read + write of {traffic_src}, scaled by heads x pairs",
                     "peak_source": f"{peaks['source']} bf16 sustained", "frac_of_burst": achieved / peaks["bf16_tflops"],
                     "frac_of_nominal_2250": achieved / 2250.0, "launch_ms": attn_avg_ms,
                     "algorithmic_flops_per_launch": comp_fl},
        "cpu_baseline": cpu,
        "kernels": {
            "attn_ms": attn_avg_ms, "merge_ms": float(np.mean(merge_ms)), "plan_ms": float(np.mean(plan_ms)),
            "merge_gbs": merge_bytes(wl, sbytes, S) / 1e9 / (float(np.mean(merge_ms)) / 1e3),
            "merge_frac_of_hbm": merge_bytes(wl, sbytes, S) / 1e9 / (float(np.mean(merge_ms)) / 1e3) / peaks["hbm_gbs"],
            "merge_frac_of_nominal_8000": merge_bytes(wl, sbytes, S) / 1e9 / (float(np.mean(merge_ms)) / 1e3) / 8000.0,
            "merge_note": "the measured peak is a plain copy (half reads, half writes); a kernel that mostly reads can exceed it",
            "plan_gbs": plan_bytes(wl, S) / 1e9 / (float(np.mean(plan_ms)) / 1e3),
            "hbm_peak_gbs": peaks["hbm_gbs"], "compose_once_ms": compose_ms,
        },
        "vs_all_compute": {"all_compute_attn_ms": full_attn_ms, "all_compute_step_ms": full_step_ms,
                           "all_compute_tflops": full_flops(wl) / 1e12 / (full_attn_ms / 1e3),
                           "all_compute_frac_of_peak": full_flops(wl) / 1e12 / (full_attn_ms / 1e3) / peak,
                           "step_time_ratio": ms_per_step / full_step_ms,
                           "full_attention_one_pass_ms": dense_ms,
                           "full_attention_one_pass_tflops": full_flops(wl) / 1e12 / (dense_ms / 1e3)},
    }
    # ---- further records of the default line, measured after the headline loop (not part of `value`)
    default_shape = (not (args.fused or args.composed or args.shard_heads) and args.group_size == 1 and args.heads is None
                     and args.state_dtype == "fp32" and args.dtype == "bf16" and args.workload == DEFAULT_WORKLOAD
                     and args.fraction is None)
    if default_shape and not args.no_extra and world == 1:
        extras = []
        extras.append(measure_config(binding, dev, wl, frac, fused=True, peaks=peaks, ctx=ctx, steps_in=steps_in))
        eps_local, ratio = ALG1_DEFAULTS[wl.name]
        extras.append(measure_alg1(binding, dev, wl, ctx, steps_in, wl.steps, eps_local, ratio))
        ctx.close()
        del steps_in, out, lse
        torch.cuda.empty_cache()
        for name, f in (("c1_cogvideox", 0.5), ("c4_hunyuan720p", 0.125)):
            extras.append(measure_config(binding, dev, inputs.WORKLOADS[name], f, peaks=peaks))
            torch.cuda.empty_cache()
        line["extra_configs"] = extras
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ further records
def _ev():
    return torch.cuda.Event(enable_timing=True)


def measure_config(binding, dev, wl, fraction, steps=5, warmup=3, fused=False, state_dtype="fp32", peaks=None, ctx=None,
                   steps_in=None):
    """One more configuration, outside the timed headline loop: anchor step + plan at `fraction`, then `steps` timed
    selective steps through dt_attn_states + dt_state_merge + dt_plan, or (fused) through dt_compose_reuse once and
    dt_attn_fused per step.  Returns a record with the kernels' times, TFLOP/s on the computed blocks, the merge's GB/s
    and the clocks sampled meanwhile."""
    sbytes = 2 if state_dtype == "bf16" else 4
    own = ctx is None
    if own:
        ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale,
                              binding.DT_STATE_BF16 if state_dtype == "bf16" else binding.DT_STATE_FP32, dev.index or 0)
        gen = inputs.StepInputs(wl, seed=0, device=dev)
        steps_in = [gen.next() for _ in range(wl.steps)]
        del gen
    stream = torch.cuda.current_stream()
    PP = wl.P * wl.P
    out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    ones = torch.ones(PP, dtype=torch.uint8, device=dev)
    masks = [torch.ones(PP, dtype=torch.uint8, device=dev), torch.ones(PP, dtype=torch.uint8, device=dev)]
    q, k, v = steps_in[0]
    ctx.dt_attn_states(q, k, v, ones, 0)
    ctx.dt_state_merge(out, lse)
    ctx.dt_plan(masks[0], target_fraction=fraction)
    comp_o = comp_l = None
    if fused:
        comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=ctx.o_state.dtype, device=dev)
        comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
        ctx.dt_compose_reuse(masks[0], comp_o, comp_l)
    torch.cuda.synchronize()
    ctx.dt_poll()
    cur, t, timers = 0, 1, []
    sampler = ClockSampler(dev.index or 0)
    for it in range(warmup + steps):
        if it == warmup:
            torch.cuda.synchronize()
            sampler.start()
        q, k, v = steps_in[1 + (t % (wl.steps - 1))] if wl.steps > 1 else steps_in[0]
        e = [_ev() for _ in range(4)]
        e[0].record(stream)
        if fused:
            ctx.dt_attn_fused(q, k, v, masks[cur], comp_o, comp_l, out, lse)
            for i in (1, 2, 3):
                e[i].record(stream)
        else:
            ctx.dt_attn_states(q, k, v, masks[cur], t)
            e[1].record(stream)
            ctx.dt_state_merge(out, lse)
            e[2].record(stream)
            ctx.dt_plan(masks[cur ^ 1], target_fraction=fraction)
            e[3].record(stream)
            cur ^= 1
        t += 1
        if it >= warmup:
            timers.append(e)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ctx.dt_poll()
    mask_np = masks[cur].cpu().numpy()
    n_comp = int((mask_np != 0).sum())
    comp_fl = computed_flops(wl, mask_np)
    attn = float(np.mean([e[0].elapsed_time(e[1]) for e in timers]))
    merge = float(np.mean([e[1].elapsed_time(e[2]) for e in timers]))
    plan = float(np.mean([e[2].elapsed_time(e[3]) for e in timers]))
    step = float(np.mean([e[0].elapsed_time(e[3]) for e in timers]))
    rec = {"workload": wl.name, "computed_pairs": n_comp, "computed_pair_fraction": n_comp / PP, "state_dtype": state_dtype,
           "step": "dt_compose_reuse once + dt_attn_fused per step" if fused else "dt_attn_states + dt_state_merge + dt_plan",
           "steps": steps, "warmup": warmup, "step_ms": step, "attn_ms": attn,
           "tflops_on_computed": comp_fl / 1e12 / (attn / 1e3),
           "effective_tflops": full_flops(wl) / 1e12 / (step / 1e3), "clocks": clocks,
           "cache_gb": wl.P * wl.B * wl.H * wl.L * (wl.D * sbytes + 4) / 1e9}
    if peaks is not None:
        rec["frac_of_sustained_peak"] = rec["tflops_on_computed"] / peaks["bf16_tflops_sustained"]
    if not fused:
        rec.update({"merge_ms": merge, "plan_ms": plan, "merge_gbs": merge_bytes(wl, sbytes) / 1e9 / (merge / 1e3)})
    if own:
        ctx.close()
    return rec


def measure_alg1(binding, dev, wl, ctx, steps_in, n_steps, eps_local, cache_ratio, host_replay=True):
    """The step loop of Algorithm 1 with the anchors decided on the device: per step dt_attn_local -> dt_planner_step ->
    dt_attn_states on the remaining COMPUTE pairs -> dt_state_merge -> dt_planner_commit (which refreshes w, alpha and
    the snapshot on anchors only).  The host reads the anchor flag and the mask after the timed region only."""
    stream = torch.cuda.current_stream()
    P = wl.P
    PP = P * P
    out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    snap_o = torch.zeros((wl.B, wl.H, wl.L, wl.D), dtype=ctx.o_state.dtype, device=dev)
    snap_l = torch.zeros((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    ctx.dt_planner_init(snap_o, snap_l, group_size=1, eps_initial=0.0, eps_local=eps_local, cache_ratio=cache_ratio)
    not_eye = (1 - torch.eye(P, dtype=torch.uint8, device=dev)).reshape(-1)
    masks = [torch.zeros(PP, dtype=torch.uint8, device=dev) for _ in range(n_steps)]
    rests = [torch.zeros(PP, dtype=torch.uint8, device=dev) for _ in range(n_steps)]
    flags = torch.zeros(n_steps, dtype=torch.int32, device=dev)
    drel = torch.zeros(n_steps, dtype=torch.float64, device=dev)
    evs = []
    sampler = ClockSampler(dev.index or 0)
    torch.cuda.synchronize()
    sampler.start()
    for t in range(n_steps):
        q, k, v = steps_in[t % len(steps_in)]
        e = [_ev() for _ in range(6)]
        e[0].record(stream)
        ctx.dt_attn_local(q, k, v, t)
        e[1].record(stream)
        ctx.dt_planner_step(masks[t], flags[t:t + 1], None, drel[t:t + 1])
        e[2].record(stream)
        torch.mul(masks[t], not_eye, out=rests[t])          # the local pairs are done already
        ctx.dt_attn_states(q, k, v, rests[t], t)
        e[3].record(stream)
        ctx.dt_state_merge(out, lse)
        e[4].record(stream)
        ctx.dt_planner_commit()
        e[5].record(stream)
        evs.append(e)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ctx.dt_poll()
    fl = flags.cpu().numpy().astype(bool)
    ms = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(5)] for e in evs])      # local, plan, rest, merge, commit
    step_ms = ms.sum(axis=1)
    frac = np.array([float(m.sum().item()) / PP for m in masks])
    planner_ms = ms[:, 1] + ms[:, 4]
    rec = {"workload": wl.name, "policy": "Algorithm 1 on the device", "eps_local": eps_local, "cache_ratio": cache_ratio,
           "steps": n_steps, "anchors": int(fl.sum()), "anchor_steps": [int(i) for i in np.nonzero(fl)[0]],
           "computed_pair_fraction_per_step": [round(float(x), 4) for x in frac],
           "mean_computed_pair_fraction": float(frac.mean()),
           "step_ms_mean": float(step_ms.mean()),
           "step_ms_anchor": float(step_ms[fl].mean()) if fl.any() else None,
           "step_ms_selective": float(step_ms[~fl].mean()) if (~fl).any() else None,
           "planner_ms_anchor": float(planner_ms[fl].mean()) if fl.any() else None,
           "planner_ms_selective": float(planner_ms[~fl].mean()) if (~fl).any() else None,
           "planner_share_of_all_compute_pass": (float(planner_ms[fl].mean() / step_ms[fl].mean()) if fl.any() else None),
           "local_drift_rel_per_step": [round(float(x), 5) for x in drel.cpu().numpy()],
           "effective_tflops": full_flops(wl) / 1e12 / (float(step_ms.mean()) / 1e3), "clocks": clocks}
    if host_replay:
        # the same sequence of plans end to end from host buffers (dt_step_host; the planner's kernels are not part of it)
        ws = torch.empty(binding.dt_step_host_workspace_bytes(ctx.cfg), dtype=torch.uint8, device=dev)
        oh = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
        lh = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        host_in = [tuple(x.cpu().pin_memory() for x in steps_in[i]) for i in range(min(2, len(steps_in)))]
        times = []
        for t in range(n_steps):
            qh, kh, vh = host_in[t % len(host_in)]
            mh = masks[t].cpu()
            t0 = time.perf_counter()
            ctx.dt_step_host(qh, kh, vh, mh, n_steps + t, oh, lh, ws)
            times.append(time.perf_counter() - t0)
        rec["e2e_step_ms_mean"] = 1e3 * float(np.mean(times[1:]))
        rec["e2e_includes"] = "dt_step_host with the recorded plan of every step: H2D q,k,v,mask + attention + merge + D2H out,lse"
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--fraction", type=float, default=None, help="target computed-pair fraction of the plan")
    ap.add_argument("--state-dtype", default="fp32", choices=["fp32", "bf16"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"], help="element type of q, k, v and the output")
    ap.add_argument("--heads", type=int, default=None,
                    help="override the head count (smaller captures under a profiler; not a bench configuration)")
    ap.add_argument("--composed", action="store_true",
                    help="compose the plan's REUSE states once after the anchor step and merge COMPUTE states + that "
                         "composed state in the selective steps (the plan then stays fixed between anchors)")
    ap.add_argument("--fused", action="store_true",
                    help="between anchors: dt_attn_fused per step (all COMPUTE slots in one pass, composed with the plan's "
                         "composed reuse state in the epilogue; no state-cache round trip, the plan stays fixed)")
    ap.add_argument("--group-size", type=int, default=1,
                    help="g >= 2: grouped state cache (ceil(P/g) + 1 slots per row; group states computed in one pass)")
    ap.add_argument("--shard-heads", action="store_true",
                    help="N > 1: the ranks share the heads of ONE layer (strong scaling; the plan's sums are all-reduced) "
                         "instead of running N independent replicas")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="leave out the extra_configs records of the default line")
    ap.add_argument("--policy", default="fraction", choices=["fraction", "alg1"],
                    help="alg1: the step loop of Algorithm 1 (anchors decided online) instead of a fixed target fraction")
    ap.add_argument("--eps-local", type=float, default=None, help="--policy alg1: anchor threshold on the local drift")
    ap.add_argument("--cache-ratio", type=float, default=None, help="--policy alg1: R, the share of units kept in the cache")
    ap.add_argument("--probe-world", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.probe_world:
        return probe_world(args)
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    wl = inputs.WORKLOADS[args.workload]
    if args.heads is not None:
        wl = dataclasses.replace(wl, H=args.heads, name=f"{wl.name}_h{args.heads}")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
