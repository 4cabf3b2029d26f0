"""GPU parity of dt_attn_fused: one pass over the keys of all COMPUTE slots, composed in the epilogue with the
composed reuse state (Eq. 2) -- against the oracle's selective step (fresh states + cached states, merged)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs
from tests.test_gpu_groups import GroupRun
from tests.test_gpu_parity import Run, check_lse, check_o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def _fused_steps(run, P, S, masks, state_dtype=torch.float32):
    """Anchor step through the cache, then for each mask: compose its REUSE states once and take fused steps."""
    wl, dev, ctx = run.wl, run.dev, run.ctx
    run.step(np.ones((P, S), np.uint8), check_states=False)
    comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=state_dtype, device=dev)
    comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    out = torch.empty_like(run.out); lse = torch.empty_like(run.lse)
    # The composed reuse state is a state of its own, stored in the cache's type: with a bf16 cache it is rounded to
    # bf16 once more (relative 2^-9 of values up to about 4, on top of the rounding of the states it was composed from
    # and of the bf16 output), so those checks allow twice the O bounds, as after an in-place group compose.
    o_scale = 2.0 if state_dtype == torch.bfloat16 else 1.0
    t = 1
    for mask in masks:
        mask = np.ascontiguousarray(mask, dtype=np.uint8).reshape(P, S)
        mask_dev = torch.from_numpy(mask.reshape(-1).copy()).to(dev)
        ctx.dt_compose_reuse(mask_dev, comp_o, comp_l)
        tc_before = ctx.dt_get_tc().copy()
        cache_before = ctx.lse_state.clone()
        for _ in range(2):                                   # the plan holds: two steps against the same composed state
            t += 1
            q, k, v = run.gen.next()
            out.fill_(float("nan")); lse.fill_(float("nan"))
            ctx.dt_attn_fused(q, k, v, mask_dev, comp_o, comp_l, out, lse)
            torch.cuda.synchronize()
            ctx.dt_poll()
            # oracle: the COMPUTE slots fresh from this step's inputs, the REUSE slots as cached at the anchor
            ses = run.ses
            saved = {bh: (ses.o[bh].copy(), ses.lse[bh].copy()) for bh in ses.o}
            saved_tc = ses.tc.copy()
            outs, lses = ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), mask, t)
            for bh in ses.o:                                 # the GPU cache was not refreshed: neither is the oracle's
                ses.o[bh], ses.lse[bh] = saved[bh]
            ses.tc = saved_tc
            out_h, lse_h = out.float().cpu().numpy(), lse.cpu().numpy()
            for (b, h), rows in run.rows.items():
                check_o(out_h[b, rows, h, :], outs[(b, h)], f"fused step {t} head {h}", scale=o_scale)
                check_lse(lse_h[b, h, rows], lses[(b, h)], f"fused step {t} head {h}")
        assert (ctx.dt_get_tc() == tc_before).all() and torch.equal(ctx.lse_state, cache_before)


def test_fused_pair_mode_config0():
    wl = inputs.WORKLOADS["c0_correctness"]
    run = Run(wl)
    # Run.step takes [P][P] masks; reuse the helper with S = P
    run.S = 4
    diag_plus = np.eye(4, dtype=np.uint8); diag_plus[0, 3] = 1; diag_plus[2, 0] = 1      # non-adjacent ranges
    _fused_steps(run, 4, 4, [inputs.banded_mask(4, 1), diag_plus, np.ones((4, 4), np.uint8)])


@pytest.mark.parametrize("D,grid,n_text,offsets,g,state_dtype", [
    (128, (4, 11, 13), 0, [0, 129, 385, 572], 1, binding.DT_STATE_FP32),
    (64, (5, 12, 13), 3, [0, 100, 300, 520, 700, 783], 3, binding.DT_STATE_FP32),     # own group with a hole
    (128, (3, 9, 11), 5, [0, 60, 100, 230, 302], 2, binding.DT_STATE_BF16),
    (64, (5, 12, 13), 3, [0, 300, 783], 1, binding.DT_STATE_BF16),                    # several 256-row query blocks
])
def test_fused_ragged(D, grid, n_text, offsets, g, state_dtype):
    wl = inputs.Workload("fused_ragged", 1, 3, D, grid, n_text, len(offsets) - 1, 2, 0.05)
    P = len(offsets) - 1
    if g == 1:
        run = Run(wl, offsets=offsets, seed=8, state_dtype=state_dtype)
        S = P
        local = np.eye(P, dtype=np.uint8)
        some = local.copy(); some[:, P - 1] = 1
    else:
        run = GroupRun(wl, g, offsets=offsets, seed=8, state_dtype=state_dtype)
        S = run.S
        local = np.zeros((P, S), np.uint8); local[:, 0] = 1
        some = local.copy(); some[:, 1] = 1
    sdt = torch.float32 if state_dtype == binding.DT_STATE_FP32 else torch.bfloat16
    _fused_steps(run, P, S, [local, some], state_dtype=sdt)


def test_fused_all_compute_without_a_composed_state_is_full_attention_and_respects_strides():
    wl = inputs.Workload("fused_full", 2, 2, 128, (3, 10, 12), 4, 3, 1, 0.05)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    q, k, v = inputs.StepInputs(wl, seed=4, device=dev).next()
    wide = torch.zeros((wl.B, wl.L, 2, wl.H, wl.D), dtype=torch.bfloat16, device=dev)
    out = wide[:, :, 1]
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    ctx.dt_attn_fused(q, k, v, torch.ones(9, dtype=torch.uint8, device=dev), None, None, out, lse)
    torch.cuda.synchronize()
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    rows = np.arange(wl.L, dtype=np.int32)
    for b in range(wl.B):
        for h in range(wl.H):
            ro, rl = orc.full_attention(qb, kb, vb, wl.scale, b, h, rows)
            check_o(out[b, :, h].float().cpu().numpy(), ro, "fused full attention")
            check_lse(lse[b, h].cpu().numpy(), rl, "fused full attention")
    assert (wide[:, :, 0] == 0).all()
    assert ctx.dt_launch_count() == 2
    with pytest.raises(binding.DitangoError):
        ctx.dt_attn_fused(q, k, v, torch.ones(9, dtype=torch.uint8, device=dev), torch.empty(1, device=dev), None, out, lse)
