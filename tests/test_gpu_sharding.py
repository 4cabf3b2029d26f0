"""Head-sharded planning (dt_plan_sums -> sum over shards -> dt_plan_from_sums) on one GPU: two contexts, each
holding half the heads of the same layer, must arrive at the mask and W that one context over all heads takes,
and at the oracle's plan.  The exchange between real ranks is an all-reduce of the same sums (covered on CPU with
gloo); here the shards' sums are added on the device."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs, sharding

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def _anchor(ctx, q, k, v, h0, h1, S):
    ones = torch.ones(ctx.cfg.P * S, dtype=torch.uint8, device=q.device)
    ctx.dt_attn_states(q[:, :, h0:h1], k[:, :, h0:h1], v[:, :, h0:h1], ones, 1)


@pytest.mark.parametrize("g", [1, 2])
@pytest.mark.parametrize("mode", ["fraction", "threshold"])
def test_two_head_shards_take_the_plan_of_all_heads(g, mode):
    wl = inputs.tiny_workload("shard", B=2, H=5, D=64, grid=(3, 10, 13), n_text=7, P=4)
    dev = torch.device("cuda", 0)
    off = wl.offsets()
    q, k, v = inputs.StepInputs(wl, seed=11, device=dev).next()
    full = binding.Context(wl.B, wl.H, wl.D, wl.L, off, wl.scale, group_size=g)
    P, S = wl.P, full.dt_num_slots()[0]
    _anchor(full, q, k, v, 0, wl.H, S)
    ranges = [sharding.head_range(wl.H, 2, r) for r in range(2)]
    assert ranges == [(0, 3), (3, 5)]
    shards = [binding.Context(wl.B, h1 - h0, wl.D, wl.L, off, wl.scale, group_size=g) for h0, h1 in ranges]
    sums = []
    for c, (h0, h1) in zip(shards, ranges):
        _anchor(c, q, k, v, h0, h1, S)
        assert torch.equal(c.lse_state, full.lse_state[:, :, h0:h1])      # same kernel, same rows: same states
        s = torch.full((P * S,), -1.0, dtype=torch.float64, device=dev)
        c.dt_plan_sums(s)
        sums.append(s)
    total = sums[0] + sums[1]
    kw = dict(target_fraction=0.5) if mode == "fraction" else dict(eps=0.2)

    def outputs():
        return (torch.zeros(P * S, dtype=torch.uint8, device=dev), torch.zeros(P * S, dtype=torch.float64, device=dev),
                torch.zeros(1, dtype=torch.float64, device=dev))

    m_full, w_full, e_full = outputs()
    full.dt_plan(m_full, w_dev=w_full, eps_out_dev=e_full, **kw)
    got = []
    for c in shards:
        m, w, e = outputs()
        c.dt_plan_from_sums(total, wl.B * wl.H, m, w_dev=w, eps_out_dev=e, **kw)
        got.append((m, w, e))
    torch.cuda.synchronize()
    for c in shards + [full]:
        c.dt_poll()
    for m, w, e in got:
        assert torch.equal(m, m_full)
        np.testing.assert_allclose(w.cpu().numpy(), w_full.cpu().numpy(), rtol=1e-12, atol=0)
        np.testing.assert_allclose(e.cpu().numpy(), e_full.cpu().numpy(), rtol=1e-12, atol=0)
    assert torch.equal(got[0][1], got[1][1])            # the same totals give the same W bit for bit on every shard
    assert 0 < int(m_full.sum()) < P * S or mode == "threshold"
    if g == 1:
        # the oracle's plan from the LSE cache of all heads (the compare and the ranking are taken in fp64 on both sides)
        W = orc.contribution(full.lse_state.double().cpu().numpy(), off)
        np.testing.assert_allclose(got[0][1].cpu().numpy().reshape(P, P), W, rtol=2e-5, atol=1e-9)
        m_orc = orc.target_fraction(W, 0.5)[0] if mode == "fraction" else orc.threshold(W, 0.2)
        assert (got[0][0].cpu().numpy().reshape(P, P) == m_orc).all()
        # the sums are what they say: W * (B * H_local * n_i) of the shard's own heads
        for s, (h0, h1) in zip(sums, ranges):
            W_r = orc.contribution(full.lse_state[:, :, h0:h1].double().cpu().numpy(), off)
            cnt = wl.B * (h1 - h0) * np.diff(off)[:, None]
            np.testing.assert_allclose(s.cpu().numpy().reshape(P, P), W_r * cnt, rtol=2e-5, atol=1e-9)


def test_one_shard_is_dt_plan_bit_for_bit_and_bad_totals_are_refused():
    wl = inputs.tiny_workload("shard1", B=1, H=3, D=128, grid=(2, 9, 11), P=3)
    dev = torch.device("cuda", 0)
    q, k, v = inputs.StepInputs(wl, seed=5, device=dev).next()
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    _anchor(ctx, q, k, v, 0, wl.H, wl.P)
    n = wl.P * wl.P
    m0, m1 = (torch.zeros(n, dtype=torch.uint8, device=dev) for _ in range(2))
    w0, w1 = (torch.zeros(n, dtype=torch.float64, device=dev) for _ in range(2))
    e0, e1 = (torch.zeros(1, dtype=torch.float64, device=dev) for _ in range(2))
    ctx.dt_plan(m0, target_fraction=0.6, w_dev=w0, eps_out_dev=e0)
    sums = torch.empty(n, dtype=torch.float64, device=dev)
    before = ctx.dt_launch_count()
    sharding.plan_sharded(ctx, wl.B * wl.H, m1, sums, target_fraction=0.6, w_dev=w1, eps_out_dev=e1)   # no process group
    assert ctx.dt_launch_count() - before == 3            # stage 1, sums, plan from sums
    torch.cuda.synchronize()
    assert torch.equal(m0, m1) and torch.equal(w0, w1) and torch.equal(e0, e1)
    with pytest.raises(binding.DitangoError):
        ctx.dt_plan_from_sums(sums, wl.B * wl.H - 1, m1)   # fewer slices than this context alone holds
    with pytest.raises(binding.DitangoError):
        ctx.dt_plan_from_sums(sums, wl.B * wl.H, m1, target_fraction=1.5)
