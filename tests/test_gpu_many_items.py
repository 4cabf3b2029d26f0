"""Persistent CTAs that walk many short work items: the start and the end of an item are where the roles of the
attention kernel hand over (first S, first P, last PV, epilogue, the next item's Q), so a protocol race shows here
first.  Each case is launched repeatedly: every launch must leave the same state cache bit for bit (the kernel has no
atomics and a fixed order of accumulation), sampled rows are compared with the oracle, and no bounded wait may
expire."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


@pytest.mark.parametrize("D,P,state_dtype,shape", [
    (64, 6, binding.DT_STATE_FP32, "short"),      # two K/V tiles per item
    (64, 12, binding.DT_STATE_BF16, "short"),     # one K/V tile per item: nothing but item starts and ends
    (128, 6, binding.DT_STATE_FP32, "short"),
    (128, 12, binding.DT_STATE_FP32, "short"),
    (64, 4, binding.DT_STATE_FP32, "wide"),       # Q, K, V larger than L2: operand loads land late
    (128, 4, binding.DT_STATE_FP32, "wide"),
])
def test_many_short_items_repeat_bit_for_bit(D, P, state_dtype, shape):
    if shape == "short":
        wl = inputs.tiny_workload("many_items", B=2, H=24, D=D, grid=(4, 16, 20), n_text=13, P=P)
    else:
        wl = inputs.tiny_workload("many_items_wide", B=1, H=48 if D == 64 else 24, D=D, grid=(10, 30, 30), n_text=0, P=P)
    dev = torch.device("cuda", 0)
    off = wl.offsets()
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, off, wl.scale, state_dtype)
    q, k, v = inputs.StepInputs(wl, seed=21, device=dev).next()
    rng = np.random.default_rng(5)
    masks = [np.ones((P, P), np.uint8)]
    for _ in range(2):
        m = (rng.random((P, P)) < 0.5).astype(np.uint8)
        np.fill_diagonal(m, 1)
        masks.append(m)
    rows = inputs.sample_rows(wl, 192, seed=3, max_heads=4)
    ses = orc.OracleSession(wl.B, wl.L, wl.H, wl.D, off, wl.scale, rows)
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    n_items = P * P * wl.B * wl.H * (-(-int(np.diff(off).max()) // 256))
    assert n_items > 8 * 148                          # several items per CTA
    for t, m in enumerate(masks):
        m_dev = torch.from_numpy(m.reshape(-1)).to(dev)
        first_o = first_l = None
        for rep in range(12):
            ctx.dt_attn_states(q, k, v, m_dev, t + 1)
            torch.cuda.synchronize()
            ctx.dt_poll()
            if rep == 0:
                first_o, first_l = ctx.o_state.clone(), ctx.lse_state.clone()
            else:
                assert torch.equal(ctx.o_state, first_o) and torch.equal(ctx.lse_state, first_l), (t, rep)
        ctx.dt_state_merge(out, lse)
        torch.cuda.synchronize()
        ref_o, ref_l = ses.step(qb, kb, vb, m, t + 1)
        for (b, h), r in rows.items():
            ridx = torch.from_numpy(r.astype(np.int64)).to(dev)
            eo = np.abs(out[b, ridx, h].float().cpu().numpy() - ref_o[(b, h)])
            el = np.abs(lse[b, h, ridx].cpu().numpy() - ref_l[(b, h)])
            assert eo.max() <= 2e-2 and eo.mean() <= 2e-3 and el.max() <= 5e-3, (t, b, h, eo.max(), el.max())
            st_l = ctx.lse_state[:, b, h][:, ridx].cpu().numpy()
            assert np.abs(st_l.T - ses.lse[(b, h)]).max() <= 5e-3
    # the one-pass mode walks the same items with longer key runs
    ones = torch.ones(P * P, dtype=torch.uint8, device=dev)
    ref = None
    for rep in range(6):
        ctx.dt_attn_fused(q, k, v, ones, None, None, out, lse)
        torch.cuda.synchronize()
        ctx.dt_poll()
        if rep == 0:
            ref = (out.clone(), lse.clone())
        else:
            assert torch.equal(out, ref[0]) and torch.equal(lse, ref[1])
