"""Head sharding of one attention layer over several GPUs, one context per GPU (one process per GPU).

The (batch, head) slices of a layer are independent in dt_attn_states and dt_state_merge, so a rank that holds
H_local of the H heads runs both on its slice with no exchange.  The plan is the one step that needs one: the
partition importance W (Eq. 8) is a mean over all heads, and every rank must take the same COMPUTE / REUSE mask
(Section 5.1.1: the strategy is the same on all devices).  Each rank therefore sums its own per-row weights
(dt_plan_sums), the P x S sums are added over the ranks by one all-reduce of doubles, and each rank finishes the
plan from the same totals (dt_plan_from_sums).  This module holds that plumbing only; every step of the
arithmetic runs in the library's kernels.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def head_range(H: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous heads [h0, h1) of `rank`: sizes differ by at most one, the first H % world ranks hold one more."""
    if not (0 <= rank < world) or H < world:
        raise ValueError(f"cannot shard {H} heads over {world} ranks (rank {rank})")
    base, extra = divmod(H, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def all_reduce_sums(sums: torch.Tensor, group=None) -> torch.Tensor:
    """Adds the ranks' sums in place (fp64; every rank ends with the same totals).  Without an initialised
    process group there is one shard and nothing to add."""
    if sums.dtype != torch.float64:
        raise TypeError("the plan's sums are exchanged as float64")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
    return sums


def plan_sharded(ctx, total_bh: int, mask_dev: torch.Tensor, sums_dev: torch.Tensor, *, eps: float = 0.0,
                 target_fraction: float = -1.0, group_size: int = 1, w_dev=None, eps_out_dev=None, group=None) -> None:
    """dt_plan over the heads of all ranks: local sums, one all-reduce, the plan from the totals.

    ctx          this rank's binding.Context (its H is the rank's share of the heads)
    total_bh     B x the number of heads over all ranks
    mask_dev     uint8 [P*S], written with the same mask on every rank
    sums_dev     float64 [P*S] scratch on this rank's device (caller-owned: nothing is allocated here)
    Runs on torch's current stream; the collective is ordered with it by torch.distributed."""
    ctx.dt_plan_sums(sums_dev)
    all_reduce_sums(sums_dev, group)
    ctx.dt_plan_from_sums(sums_dev, total_bh, mask_dev, eps=eps, target_fraction=target_fraction, group_size=group_size,
                          w_dev=w_dev, eps_out_dev=eps_out_dev)
