"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs.  Tolerances are the ones stated for bf16 inputs with fp32 accumulation:
O max-abs <= 2e-2 and mean-abs <= 2e-3, LSE abs <= 5e-3, plan mask bit-exact."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

O_MAX, O_MEAN, LSE_ABS = 2e-2, 2e-3, 5e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def check_o(got, ref, what="", scale=1.0):
    """scale > 1 only where states of a bf16 cache have been composed into a state that is stored again (in place by
    dt_group_compose, or as the composed reuse state that dt_attn_fused reads): every such composition rounds the state
    to bf16 once more (relative 2^-9 of values up to about 4), on top of the rounding of the stored states."""
    err = np.abs(np.asarray(got, dtype=np.float64) - ref)
    assert err.max() <= scale * O_MAX, f"{what}: O max abs err {err.max():.3e}"
    assert err.mean() <= scale * O_MEAN, f"{what}: O mean abs err {err.mean():.3e}"


def check_lse(got, ref, what=""):
    err = np.abs(np.asarray(got, dtype=np.float64) - ref)
    assert err.max() <= LSE_ABS, f"{what}: LSE max abs err {err.max():.3e}"


class Run:
    """Drives one workload through the C ABI and the oracle side by side."""

    def __init__(self, wl, rows_by_bh=None, state_dtype=binding.DT_STATE_FP32, seed=0, offsets=None, fp16=False):
        self.wl = wl
        self.off = wl.offsets() if offsets is None else np.asarray(offsets, dtype=np.int32)
        self.P = self.off.size - 1
        self.dev = torch.device("cuda", 0)
        in_dt = torch.float16 if fp16 else torch.bfloat16
        self.ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, self.off, wl.scale, state_dtype, 0,
                                   input_dtype=binding.DT_INPUT_FP16 if fp16 else binding.DT_INPUT_BF16)
        self.gen = inputs.StepInputs(wl, seed=seed, device=self.dev, dtype=in_dt)
        if rows_by_bh is None:
            rows_by_bh = {(b, h): np.arange(wl.L, dtype=np.int32) for b in range(wl.B) for h in range(wl.H)}
        self.rows = rows_by_bh
        self.ses = orc.OracleSession(wl.B, wl.L, wl.H, wl.D, self.off, wl.scale, rows_by_bh, fp16=fp16)
        self.out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=in_dt, device=self.dev)
        self.lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=self.dev)
        self.t = 0

    def step(self, mask, check_states=False):
        self.t += 1
        q, k, v = self.gen.next()
        mask = np.ascontiguousarray(mask, dtype=np.uint8).reshape(self.P, self.P)
        mask_dev = torch.from_numpy(mask).to(self.dev)
        self.ctx.dt_attn_states(q, k, v, mask_dev, self.t)
        self.ctx.dt_state_merge(self.out, self.lse)
        torch.cuda.synchronize()
        self.ctx.dt_poll()
        qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
        outs, lses = self.ses.step(qb, kb, vb, mask, self.t)
        out_h = self.out.float().cpu().numpy()
        lse_h = self.lse.cpu().numpy()
        for (b, h), rows in self.rows.items():
            check_o(out_h[b, rows, h, :], outs[(b, h)], f"step {self.t} head {h} merged")
            check_lse(lse_h[b, h, rows], lses[(b, h)], f"step {self.t} head {h} merged")
        if check_states:
            o_st = self.ctx.o_state.float().cpu().numpy()     # [P, B, H, L, D]
            l_st = self.ctx.lse_state.cpu().numpy()           # [P, B, H, L]
            for (b, h), rows in self.rows.items():
                for j in range(self.P):
                    check_o(o_st[j, b, h, rows, :], self.ses.o[(b, h)][:, j, :], f"step {self.t} state j={j}")
                    check_lse(l_st[j, b, h, rows], self.ses.lse[(b, h)][:, j], f"step {self.t} state j={j}")
        assert (self.ctx.dt_get_tc() == self.ses.tc).all()
        return q, k, v


def test_config0_two_steps_full_then_banded():
    """Correctness config: 1024 tokens, 2 heads, D = 64, P = 4; step 1 computes all 16 pairs, step 2
    computes |i-j| <= 1 and reuses the rest from step 1.  Every pair state and the merged output are
    compared element by element."""
    wl = inputs.WORKLOADS["c0_correctness"]
    run = Run(wl)
    run.step(np.ones((4, 4), np.uint8), check_states=True)
    run.step(inputs.banded_mask(4, 1), check_states=True)
    assert run.ctx.dt_launch_count() == 6


@pytest.mark.parametrize("D,grid,n_text,offsets", [
    (64, (2, 6, 7), 0, [0, 30, 61, 84]),                 # partitions smaller than one tile
    (128, (3, 9, 11), 5, [0, 100, 302]),                 # ragged tail inside a 128-row tile, text rows
    (128, (4, 11, 13), 0, [0, 129, 385, 572]),           # 1 / 2 / 1.46 tiles
    (64, (5, 12, 13), 3, [0, 300, 783]),                 # more than one 256-row query block per partition
])
def test_ragged_partitions_and_tails(D, grid, n_text, offsets):
    wl = inputs.Workload("ragged", 1, 3, D, grid, n_text, len(offsets) - 1, 2, 0.05)
    assert wl.L == offsets[-1]
    P = len(offsets) - 1
    run = Run(wl, offsets=offsets, seed=5)
    run.step(np.ones((P, P), np.uint8), check_states=True)
    run.step(np.eye(P, dtype=np.uint8), check_states=True)


@pytest.mark.parametrize("D", [64, 128])
def test_query_tiles_pair_across_partitions(D):
    """The attention kernel's work items are pairs of 128-row query tiles that attend to the same KV partition, taken
    from all query partitions that compute it: partitions of 3, 1, 5 and 2 tiles (the last ones ragged) make items whose
    two tiles belong to different query partitions, under masks that leave columns with one, several or all of them.
    Every pair state and the merged output, element by element."""
    offsets = [0, 300, 420, 1000, 1190]                  # 300, 120, 580, 190 rows: 3, 1, 5, 2 tiles
    wl = inputs.Workload("tilepairs", 1, 2, D, (2, 17, 35), 0, 4, 3, 0.05)
    assert wl.L == offsets[-1]
    run = Run(wl, offsets=offsets, seed=8)
    run.step(np.ones((4, 4), np.uint8), check_states=True)
    run.step(np.array([[1, 0, 1, 0], [1, 1, 0, 0], [0, 1, 1, 1], [1, 0, 0, 1]], np.uint8), check_states=True)
    run.step(np.eye(4, dtype=np.uint8), check_states=True)


def test_batch_two_and_bf16_state_cache():
    wl = inputs.Workload("b2", 2, 2, 128, (2, 10, 13), 0, 2, 2, 0.05)
    run = Run(wl, state_dtype=binding.DT_STATE_BF16, seed=2)
    run.step(np.ones((2, 2), np.uint8), check_states=True)
    run.step(np.array([[1, 0], [1, 1]], np.uint8), check_states=True)


def test_strided_inputs_and_output():
    """Q, K, V packed as one [B, L, 3, H, D] buffer (strides are not the contiguous ones)."""
    wl = inputs.Workload("strided", 1, 2, 64, (2, 8, 9), 0, 2, 1, 0.05)
    dev = torch.device("cuda", 0)
    q, k, v = inputs.StepInputs(wl, seed=7, device=dev).next()
    packed = torch.stack([q, k, v], dim=2).contiguous()
    qs, ks, vs = packed[:, :, 0], packed[:, :, 1], packed[:, :, 2]
    assert not qs.is_contiguous()
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    ones = torch.ones(4, dtype=torch.uint8, device=dev)
    out_wide = torch.zeros((wl.B, wl.L, 2, wl.H, wl.D), dtype=torch.bfloat16, device=dev)
    out = out_wide[:, :, 1]
    ctx.dt_attn_states(qs, ks, vs, ones, 1)
    ctx.dt_state_merge(out, None)
    torch.cuda.synchronize()
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    for h in range(wl.H):
        ref, _ = orc.full_attention(qb, kb, vb, wl.scale, 0, h, np.arange(wl.L, dtype=np.int32))
        check_o(out[0, :, h].float().cpu().numpy(), ref, "strided")
    assert (out_wide[:, :, 0] == 0).all()


def test_state_merge_alone_on_oracle_states():
    """dt_state_merge fed with states produced by the oracle (uploaded), against the oracle's merge."""
    rng = np.random.default_rng(3)
    B, H, D, L, P = 1, 3, 128, 77, 5
    off = orc.uniform_offsets(L, P)
    o_st = rng.standard_normal((P, B, H, L, D))
    l_st = rng.standard_normal((P, B, H, L)) * 4.0
    l_st[2, 0, 1, 5] = -np.inf                       # a state without mass has weight zero
    dev = torch.device("cuda", 0)
    for sdt, tdt in ((binding.DT_STATE_FP32, torch.float32), (binding.DT_STATE_BF16, torch.bfloat16)):
        ctx = binding.Context(B, H, D, L, off, 0.1, sdt, alloc_cache=False)
        o_dev = torch.from_numpy(o_st).to(tdt).to(dev)
        l_dev = torch.from_numpy(l_st).to(torch.float32).to(dev)
        ctx.dt_bind_cache(o_dev, l_dev)
        out = torch.empty((B, L, H, D), dtype=torch.bfloat16, device=dev)
        lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
        ctx.dt_state_merge(out, lse)
        torch.cuda.synchronize()
        o_in = o_dev.double().cpu().numpy()              # what the kernel actually read
        l_in = l_dev.double().cpu().numpy()
        ref_o, ref_l = orc.merge(np.moveaxis(o_in, 0, 3).reshape(B * H * L, P, D),
                                 np.moveaxis(l_in, 0, 3).reshape(B * H * L, P))
        got = out.float().cpu().numpy().transpose(0, 2, 1, 3).reshape(B * H * L, D)
        check_o(got, ref_o, "merge alone")
        check_lse(lse.cpu().numpy().reshape(-1), ref_l, "merge alone")


@pytest.mark.parametrize("state_dtype", [binding.DT_STATE_FP32, binding.DT_STATE_BF16])
def test_composed_reuse_state_and_planned_merge(state_dtype):
    """Fig. 6 / Eq. 15: the REUSE states of a plan are composed once into one cached state per row; a
    selective step then merges its COMPUTE states with that composed state.  The composed state is
    compared with the oracle's composition of the same slots, the planned merge with the oracle's
    step output (which composes all P slots), over uneven partitions and a block that straddles them."""
    offsets = [0, 100, 257, 300, 521, 700]
    wl = inputs.Workload("compose", 1, 2, 128, (4, 7, 25), 0, 5, 2, 0.05)
    P = 5
    run = Run(wl, offsets=offsets, seed=13, state_dtype=state_dtype)
    run.step(np.ones((P, P), np.uint8))
    mask = inputs.banded_mask(P, 1)
    mask[4, 0] = 1                                        # a non-banded COMPUTE pair
    mask[2, :] = 1                                        # a query partition without any REUSE slot
    dev = run.dev
    mask_dev = torch.from_numpy(mask.reshape(-1).copy()).to(dev)
    sdt = torch.float32 if state_dtype == binding.DT_STATE_FP32 else torch.bfloat16
    comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=sdt, device=dev)
    comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    run.ctx.dt_compose_reuse(mask_dev, comp_o, comp_l)
    torch.cuda.synchronize()
    run.ctx.dt_poll()
    part = np.searchsorted(np.asarray(offsets), np.arange(wl.L), side="right") - 1
    for (b, h), rows in run.rows.items():
        o_ref = np.zeros((wl.L, wl.D)); l_ref = np.full(wl.L, -np.inf)
        for i in range(P):
            sel = np.nonzero(part == i)[0]
            reuse = [j for j in range(P) if mask[i, j] == 0]
            if reuse:
                o_ref[sel], l_ref[sel] = orc.merge(run.ses.o[(b, h)][sel][:, reuse, :], run.ses.lse[(b, h)][sel][:, reuse])
        got_l = comp_l[b, h].cpu().numpy()
        fin = np.isfinite(l_ref)
        assert (np.isneginf(got_l) == ~fin).all()
        check_lse(got_l[fin], l_ref[fin], "composed state")
        check_o(comp_o[b, h].float().cpu().numpy(), o_ref, "composed state")
    # selective step: fresh COMPUTE states, then COMPUTE slots (+) composed state
    run.t += 1
    q, k, v = run.gen.next()
    run.ctx.dt_attn_states(q, k, v, mask_dev, run.t)
    out2 = torch.empty_like(run.out); lse2 = torch.empty_like(run.lse)
    run.ctx.dt_state_merge_planned(mask_dev, comp_o, comp_l, out2, lse2)
    run.ctx.dt_state_merge(run.out, run.lse)
    torch.cuda.synchronize()
    run.ctx.dt_poll()
    outs, lses = run.ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), mask, run.t)
    for (b, h), rows in run.rows.items():
        check_o(out2[b, :, h].float().cpu().numpy(), outs[(b, h)], "planned merge")
        check_lse(lse2[b, h].cpu().numpy(), lses[(b, h)], "planned merge")
    assert (out2.float() - run.out.float()).abs().max().item() <= 2e-2
    assert (lse2 - run.lse).abs().max().item() <= 5e-3


def test_planned_merge_with_sixteen_partitions_odd_rows_per_block():
    """P = 16 with fp32 states gives 17 sources and 7 rows per block in the planned merge: the shared
    memory carve-up (tiles, LSEs, mbarrier) must stay aligned for every such combination."""
    wl = inputs.Workload("p16", 1, 1, 128, (1, 16, 41), 0, 16, 2, 0.05)      # 656 tokens, 41 per partition
    run = Run(wl, seed=17)
    run.step(np.ones((16, 16), np.uint8))
    mask = inputs.banded_mask(16, 2)
    dev = run.dev
    mask_dev = torch.from_numpy(mask.reshape(-1).copy()).to(dev)
    comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=torch.float32, device=dev)
    comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    run.ctx.dt_compose_reuse(mask_dev, comp_o, comp_l)
    run.t += 1
    q, k, v = run.gen.next()
    run.ctx.dt_attn_states(q, k, v, mask_dev, run.t)
    run.ctx.dt_state_merge_planned(mask_dev, comp_o, comp_l, run.out, run.lse)
    torch.cuda.synchronize()
    run.ctx.dt_poll()
    outs, lses = run.ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), mask, run.t)
    check_o(run.out[0, :, 0].float().cpu().numpy(), outs[(0, 0)], "planned merge P=16")
    check_lse(run.lse[0, 0].cpu().numpy(), lses[(0, 0)], "planned merge P=16")


def _plan_case(wl, lse_host, off, fractions, eps_list):
    """dt_plan on a given LSE cache (fp32 values) against the oracle fed the same values."""
    dev = torch.device("cuda", 0)
    P = off.size - 1
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, off, wl.scale, alloc_cache=False)
    o_dummy = torch.empty((P, wl.B, wl.H, wl.L, wl.D), dtype=torch.float32, device=dev)
    l_dev = torch.from_numpy(lse_host.astype(np.float32)).to(dev)
    ctx.dt_bind_cache(o_dummy, l_dev)
    W_ref = orc.contribution(lse_host.astype(np.float32).astype(np.float64), off)
    mask = torch.empty(P * P, dtype=torch.uint8, device=dev)
    W = torch.empty(P * P, dtype=torch.float64, device=dev)
    eps_out = torch.empty(1, dtype=torch.float64, device=dev)
    for f in fractions:
        ctx.dt_plan(mask, target_fraction=f, w_dev=W, eps_out_dev=eps_out)
        torch.cuda.synchronize()
        Wg = W.cpu().numpy().reshape(P, P)
        np.testing.assert_allclose(Wg, W_ref, rtol=2e-5, atol=1e-9)
        np.testing.assert_allclose(Wg.sum(1), 1.0, atol=1e-5)
        ref_mask, ref_eps, K = orc.target_fraction(W_ref, f)
        # the decision itself, taken on the GPU's own W in the same precision, must be reproduced exactly
        own_mask, own_eps, _ = orc.target_fraction(Wg, f)
        got = mask.cpu().numpy().reshape(P, P)
        assert (got == own_mask).all() and eps_out.item() == own_eps
        assert got.sum() == K
        # and it equals the oracle's plan whenever the oracle's own margin is resolvable in fp32
        offd = ~np.eye(P, dtype=bool)
        rel = np.abs(W_ref - ref_eps) / max(ref_eps, 1e-300)
        decidable = (rel > 1e-4) | ~offd            # pairs the fp32 measure can decide; the rest are reported by name
        gap = rel[offd].min()
        print(f"[plan margin] {wl.name} f={f}: min |W - eps| / eps = {gap:.3e} -> "
              + ("well-conditioned" if gap > 1e-4 else f"ILL-CONDITIONED ({int((~decidable).sum())} pairs undecidable)"))
        assert (got == ref_mask)[decidable].all()
        if gap > 1e-4:
            assert eps_out.item() == pytest.approx(ref_eps, rel=1e-4)
    for eps in eps_list:
        ctx.dt_plan(mask, eps=eps, w_dev=W, eps_out_dev=eps_out)
        torch.cuda.synchronize()
        Wg = W.cpu().numpy().reshape(P, P)
        got = mask.cpu().numpy().reshape(P, P)
        assert (got == orc.threshold(Wg, eps)).all() and eps_out.item() == eps
        if (np.abs(W_ref - eps)[~np.eye(P, dtype=bool)].min() / eps) > 1e-4:
            assert (got == orc.threshold(W_ref, eps)).all()
    # run-to-run bit reproducibility (no atomics in the reduction)
    W2 = torch.empty_like(W)
    ctx.dt_plan(mask, eps=0.1, w_dev=W2)
    torch.cuda.synchronize()
    assert torch.equal(W, W2)


def test_plan_on_synthetic_lse_uneven_partitions():
    rng = np.random.default_rng(4)
    wl = inputs.Workload("plan", 2, 3, 64, (1, 1, 2500), 0, 5, 1, 0.05)
    off = np.array([0, 100, 1300, 1301, 2400, 2500], np.int32)
    P = 5
    dist = np.abs(np.subtract.outer(np.arange(P), np.arange(P)))
    part = np.searchsorted(off, np.arange(wl.L), side="right") - 1
    lse = rng.standard_normal((P, wl.B, wl.H, wl.L)) * 0.5
    for j in range(P):
        lse[j] += -1.1 * dist[part, j]
    _plan_case(wl, lse, off, [0.0, 0.2, 0.4, 0.52, 0.8, 1.0], [0.05, 0.2, 0.5])


@pytest.mark.parametrize("P,g", [(8, 2), (8, 4), (12, 5), (32, 8), (6, 6)])
def test_grouped_plan_matches_oracle_rule(P, g):
    """dt_plan_grouped against the oracle's group rule applied to the GPU's own W (same fp64 decision),
    in threshold and target-fraction mode, for group sizes that do and do not divide P."""
    rng = np.random.default_rng(100 + P + g)
    L = 40 * P
    wl = inputs.Workload("grp", 1, 2, 64, (1, 1, L), 0, P, 1, 0.05)
    off = wl.offsets()
    dev = torch.device("cuda", 0)
    part = np.searchsorted(off, np.arange(L), side="right") - 1
    dist = np.abs(np.subtract.outer(np.arange(P), np.arange(P)))
    lse = rng.standard_normal((P, wl.B, wl.H, L)) * 0.6
    for j in range(P):
        lse[j] += -0.7 * dist[part, j]
    ctx = binding.Context(wl.B, wl.H, wl.D, L, off, wl.scale, alloc_cache=False)
    ctx.dt_bind_cache(torch.empty((P, wl.B, wl.H, L, wl.D), device=dev), torch.from_numpy(lse.astype(np.float32)).to(dev))
    mask = torch.empty(P * P, dtype=torch.uint8, device=dev)
    W = torch.empty(P * P, dtype=torch.float64, device=dev)
    eps_out = torch.empty(1, dtype=torch.float64, device=dev)
    for f in (0.0, 0.25, 0.4, 0.7, 1.0):
        ctx.dt_plan_grouped(mask, g, target_fraction=f, w_dev=W, eps_out_dev=eps_out)
        torch.cuda.synchronize()
        Wg = W.cpu().numpy().reshape(P, P)
        ref_mask, ref_eps, n = orc.group_plan(Wg, g, target_fraction=f)
        got = mask.cpu().numpy().reshape(P, P)
        assert (got == ref_mask).all() and got.sum() == n and eps_out.item() == ref_eps
    for eps in (0.02, 0.1, 0.3):
        ctx.dt_plan_grouped(mask, g, eps=eps, w_dev=W, eps_out_dev=eps_out)
        torch.cuda.synchronize()
        Wg = W.cpu().numpy().reshape(P, P)
        ref_mask, _, _ = orc.group_plan(Wg, g, eps=eps)
        assert (mask.cpu().numpy().reshape(P, P) == ref_mask).all() and eps_out.item() == eps


def test_plan_threshold_equality_is_reuse():
    """W exactly equal to eps must give REUSE (strict '>'): constant LSEs give W = 1/P exactly."""
    wl = inputs.Workload("eq", 1, 1, 64, (1, 1, 64), 0, 4, 1, 0.05)
    off = wl.offsets()
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, off, wl.scale, alloc_cache=False)
    ctx.dt_bind_cache(torch.empty((4, 1, 1, 64, 64), device=dev), torch.zeros((4, 1, 1, 64), device=dev))
    mask = torch.empty(16, dtype=torch.uint8, device=dev)
    ctx.dt_plan(mask, eps=0.25)
    assert (mask.cpu().numpy().reshape(4, 4) == np.eye(4)).all()
    ctx.dt_plan(mask, eps=0.2499999)
    assert mask.cpu().numpy().all()


def test_plan_from_gpu_states_of_config0_matches_oracle_plan():
    """End of an anchor step: dt_plan on the cache dt_attn_states just filled, against the oracle's
    plan from the oracle's own LSEs (f = 0.5), and the plan then drives the next step."""
    wl = inputs.WORKLOADS["c0_correctness"]
    run = Run(wl)
    run.step(np.ones((4, 4), np.uint8))
    dev = run.dev
    mask = torch.empty(16, dtype=torch.uint8, device=dev)
    W = torch.empty(16, dtype=torch.float64, device=dev)
    run.ctx.dt_plan(mask, target_fraction=0.5, w_dev=W)
    torch.cuda.synchronize()
    lse_ref = np.empty((4, wl.B, wl.H, wl.L))
    for (b, h), rows in run.rows.items():
        lse_ref[:, b, h, :] = run.ses.lse[(b, h)].T
    W_ref = orc.contribution(lse_ref, run.off)
    np.testing.assert_allclose(W.cpu().numpy().reshape(4, 4), W_ref, rtol=1e-3, atol=1e-6)
    ref_mask, ref_eps, K = orc.target_fraction(W_ref, 0.5)
    got = mask.cpu().numpy().reshape(4, 4)
    assert K == 8 and got.sum() == 8
    assert (got == ref_mask).all()
    run.step(got, check_states=True)


def test_reuse_of_never_computed_pair_is_reported():
    wl = inputs.tiny_workload(grid=(2, 6, 7), P=3)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    q, k, v = inputs.StepInputs(wl, device=dev).next()
    ctx.dt_attn_states(q, k, v, torch.eye(3, dtype=torch.uint8, device=dev).reshape(-1).contiguous(), 0)
    with pytest.raises(binding.DitangoError) as ei:
        ctx.dt_poll()
    assert ei.value.status == binding.DT_ERR_STATE
    ctx.dt_poll()                                            # cleared by the first poll
    tc = ctx.dt_get_tc()
    assert (tc.diagonal() == 0).all() and tc[0, 1] == -1
    # snapshot / resume of t_c
    tc2 = tc.copy(); tc2[0, 1] = 5
    ctx.dt_set_tc(tc2)
    assert (ctx.dt_get_tc() == tc2).all()


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A wait that nothing will ever satisfy runs out after its limit, is reported by dt_poll as
    DT_ERR_TIMEOUT, and the same context then runs a normal step."""
    wl = inputs.tiny_workload(grid=(2, 6, 7), P=3)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    ctx.dt_selftest_wait_timeout(limit_us=500)
    with pytest.raises(binding.DitangoError) as ei:
        ctx.dt_poll()
    assert ei.value.status == binding.DT_ERR_TIMEOUT
    ctx.dt_poll()                                            # cleared
    q, k, v = inputs.StepInputs(wl, device=dev).next()
    out = torch.empty_like(q)
    ctx.dt_attn_states(q, k, v, torch.ones(9, dtype=torch.uint8, device=dev), 0)
    ctx.dt_state_merge(out, None)
    torch.cuda.synchronize()
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    ref, _ = orc.full_attention(qb, kb, vb, wl.scale, 0, 1, np.arange(wl.L, dtype=np.int32))
    check_o(out[0, :, 1].float().cpu().numpy(), ref, "after self-test")


def test_argument_errors_do_not_launch():
    wl = inputs.tiny_workload()
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale, alloc_cache=False)
    q, k, v = inputs.StepInputs(wl, device=dev).next()
    mask = torch.ones(9, dtype=torch.uint8, device=dev)
    with pytest.raises(binding.DitangoError) as ei:
        ctx.dt_attn_states(q, k, v, mask, 1)                 # cache not bound
    assert ei.value.status == binding.DT_ERR_STATE
    with pytest.raises(binding.DitangoError) as ei:
        ctx.dt_bind_cache(torch.empty(16, device=dev), torch.empty(16, device=dev))   # too small
    assert ei.value.status == binding.DT_ERR_STATE
    assert ctx.dt_launch_count() == 0


def test_step_from_host_buffers():
    wl = inputs.Workload("host", 1, 2, 64, (2, 9, 10), 0, 2, 1, 0.05)
    q, k, v = inputs.StepInputs(wl, seed=9, device="cpu").next()
    qp, kp, vp = (x.contiguous().pin_memory() for x in (q, k, v))
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale)
    ws = torch.empty(binding.dt_step_host_workspace_bytes(ctx.cfg), dtype=torch.uint8, device="cuda:0")
    out = torch.empty_like(q).pin_memory()
    lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32).pin_memory()
    mask = torch.ones(4, dtype=torch.uint8)
    ctx.dt_step_host(qp, kp, vp, mask, 1, out, lse, ws)
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    for h in range(wl.H):
        ref, ref_l = orc.full_attention(qb, kb, vb, wl.scale, 0, h, np.arange(wl.L, dtype=np.int32))
        check_o(out[0, :, h].float().numpy(), ref, "host step")
        check_lse(lse[0, h].numpy(), ref_l, "host step")


def test_algorithm1_planner_over_denoising_steps():
    """Algorithm 1 on the device over several steps (local attention -> plan -> remaining pairs -> merge ->
    commit), against the oracle's planner rule.  The decision is taken in fp64 on both sides from the GPU's
    own w, alpha and local drift (recomputed on the host in fp64 from the GPU's cache and snapshot); w and
    alpha themselves are compared with the oracle's values from the oracle's states."""
    wl = inputs.Workload("alg1", 1, 2, 64, (4, 16, 16), 0, 4, 6, 0.05)
    P, g, R, eps_local = 4, 1, 0.5, 0.5
    run = Run(wl, seed=21)
    dev, ctx, off = run.dev, run.ctx, run.off
    snap_o = torch.zeros((wl.B, wl.H, wl.L, wl.D), dtype=torch.float32, device=dev)
    snap_l = torch.zeros((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    ctx.dt_planner_init(snap_o, snap_l, group_size=g, eps_initial=0.0, eps_local=eps_local, cache_ratio=R)
    mask = torch.zeros(P * P, dtype=torch.uint8, device=dev)
    flag = torch.zeros(1, dtype=torch.int32, device=dev)
    ase = torch.zeros(P * P, dtype=torch.float64, device=dev)
    drel = torch.zeros(1, dtype=torch.float64, device=dev)
    part = np.searchsorted(off, np.arange(wl.L), side="right") - 1
    eps, have_anchor = 0.0, False
    anchors, selective = 0, 0
    anchor_local = None          # the oracle's local states of the last anchor: {(b, h, i): (OUT, LSE)}
    for t in range(wl.steps):
        q, k, v = run.gen.next()
        ctx.dt_attn_local(q, k, v, t)                              # local states of the step
        ctx.dt_planner_step(mask, flag, ase, drel)
        torch.cuda.synchronize()
        # --- the device's drift (Eq. 10's norm, Eq. 14's relative drift) against the oracle's own states: the local
        # states of this step by Eq. 1 from the same inputs, the anchor's kept from the step that was one
        qb_, kb_, vb_ = (inputs.bf16_bits(x) for x in (q, k, v))
        local_now = {}
        for b_ in range(wl.B):
            for h_ in range(wl.H):
                for i in range(P):
                    rows_i = np.arange(off[i], off[i + 1], dtype=np.int32)
                    local_now[(b_, h_, i)] = orc.pair_state(qb_, kb_, vb_, wl.scale, b_, h_, rows_i, int(off[i]), int(off[i + 1]))
        if anchor_local is not None:
            d_or = sum(orc.state_norm_sq(local_now[key][0] - anchor_local[key][0], local_now[key][1] - anchor_local[key][1])
                       for key in local_now)
            b_or = sum(orc.state_norm_sq(*anchor_local[key]) for key in local_now)
            assert drel.item() == pytest.approx(np.sqrt(d_or / b_or), rel=3e-2), t
        # --- the oracle rule on the GPU's own quantities
        w_g, alpha_g, eps_before, have_g = ctx.dt_planner_get()
        assert have_g == have_anchor
        o_c = ctx.o_state.double().cpu().numpy(); l_c = ctx.lse_state.double().cpu().numpy()
        so = snap_o.double().cpu().numpy(); sl = snap_l.double().cpu().numpy()
        drift = np.zeros(P); base = np.zeros(P)
        for i in range(P):
            rows = part == i
            drift[i] = ((o_c[i][:, :, rows] - so[:, :, rows]) ** 2).sum() + ((l_c[i][:, :, rows] - sl[:, :, rows]) ** 2).sum()
            base[i] = (so[:, :, rows] ** 2).sum() + (sl[:, :, rows] ** 2).sum()
        # eps_before already holds the updated value if this step is an anchor; the rule is applied with the
        # value the device used, which the test tracks itself
        ref = orc.planner_step(w_g, alpha_g, drift, base, g, eps, eps_local, R, have_anchor)
        got_mask = mask.cpu().numpy().reshape(P, P)
        assert bool(flag.item()) == ref["is_anchor"], (t, ref["delta_rel"])
        assert (got_mask == ref["mask"]).all(), t
        if have_anchor:
            np.testing.assert_allclose(ase.cpu().numpy().reshape(P, P)[~np.eye(P, dtype=bool)],
                                       ref["ase"][~np.eye(P, dtype=bool)], rtol=1e-4)
            assert drel.item() == pytest.approx(ref["delta_rel"], rel=1e-4)
            valid = ref["ase"][~np.isnan(ref["ase"])]
            if not ref["is_anchor"]:                              # margin of the decision w.r.t. fp32 partial sums
                assert (np.abs(valid - eps) / max(eps, 1e-300)).min() > 1e-5
        assert eps_before == pytest.approx(ref["eps"], rel=1e-4)
        eps = eps_before
        # --- the rest of the step
        rest = torch.from_numpy((got_mask * (1 - np.eye(P, dtype=np.uint8))).reshape(-1).copy()).to(dev)
        ctx.dt_attn_states(q, k, v, rest, t)
        ctx.dt_state_merge(run.out, run.lse)
        ctx.dt_planner_commit()
        torch.cuda.synchronize()
        ctx.dt_poll()
        outs, lses = run.ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), got_mask, t)
        for (b, h), rows in run.rows.items():
            check_o(run.out[b, :, h].float().cpu().numpy(), outs[(b, h)], f"alg1 step {t}")
            check_lse(run.lse[b, h].cpu().numpy(), lses[(b, h)], f"alg1 step {t}")
        assert (ctx.dt_get_tc() == run.ses.tc).all()
        if ref["is_anchor"]:
            anchors += 1
            have_anchor = True
            anchor_local = local_now
            # w (Eq. 8) and alpha (Eq. 9) against the oracle's states of this anchor
            w_g, alpha_g, _, _ = ctx.dt_planner_get()
            lse_ref = np.empty((P, wl.B, wl.H, wl.L)); nsq = np.zeros((P, P))
            for (b, h), rows in run.rows.items():
                lse_ref[:, b, h, :] = run.ses.lse[(b, h)].T
                for i in range(P):
                    sel = part == i
                    for j in range(P):
                        nsq[i, j] += orc.state_norm_sq(run.ses.o[(b, h)][sel, j, :], run.ses.lse[(b, h)][sel, j])
            np.testing.assert_allclose(w_g, orc.contribution(lse_ref, off), rtol=2e-3, atol=1e-6)
            np.testing.assert_allclose(alpha_g, orc.scale_ratios(nsq), rtol=2e-3)
            assert torch.equal(snap_l, torch.stack([ctx.lse_state[i] for i in range(P)])[torch.from_numpy(part).to(dev), :, :, torch.arange(wl.L, device=dev)].permute(1, 2, 0))
        else:
            selective += 1
            assert 0 < got_mask.sum() < P * P
    assert anchors >= 2 and selective >= 1


@pytest.mark.parametrize("D,fp16", [(128, False), (64, False), (128, True)])
def test_growing_logits_move_the_reference_maximum(D, fp16):
    """Logits that grow along the key axis by far more than the rescale threshold (and by more than fp32's exponent
    range in total), plus rows whose largest logit sits in the first tile: the stale-reference softmax has to move
    its reference (and rescale O and l) again and again, and must never overflow."""
    B, H, L, P = 1, 2, 1100, 2
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(17)
    dt = torch.float16 if fp16 else torch.bfloat16
    q = rng.standard_normal((B, L, H, D)).astype(np.float32)
    k = rng.standard_normal((B, L, H, D)).astype(np.float32) * 0.1
    v = rng.standard_normal((B, L, H, D)).astype(np.float32)
    ramp = np.linspace(0.0, 1.0, L, dtype=np.float32)
    # head 0: k aligned with a fixed direction u with a coefficient that rises along the keys; q rows aligned with +u
    # (logits rise to about +300 in natural units at the last key) or -u (largest logit at the first key)
    u = np.zeros(D, np.float32); u[:8] = 1.0 / np.sqrt(8.0)
    k[0, :, 0, :] += np.outer(ramp * 30.0, u)
    sign = np.where(np.arange(L) % 3 == 0, -1.0, 1.0).astype(np.float32)
    q[0, :, 0, :] = np.outer(sign * 10.0, u) + 0.1 * q[0, :, 0, :]
    qt, kt, vt = (torch.from_numpy(x).to(dt).to(dev) for x in (q, k, v))
    scale = 1.0
    off = np.array([0, 500, L], dtype=np.int32)
    ctx = binding.Context(B, H, D, L, off, scale, input_dtype=binding.DT_INPUT_FP16 if fp16 else binding.DT_INPUT_BF16)
    out = torch.empty((B, L, H, D), dtype=dt, device=dev)
    lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
    ctx.dt_attn_states(qt, kt, vt, torch.ones(P * P, dtype=torch.uint8, device=dev), 0)
    ctx.dt_state_merge(out, lse)
    torch.cuda.synchronize()
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (qt, kt, vt))
    rows = np.arange(L, dtype=np.int32)
    lse_max = -np.inf
    for h in range(H):
        ro, rl = orc.full_attention(qb, kb, vb, scale, 0, h, rows, fp16=fp16)
        lse_max = max(lse_max, rl.max())
        assert np.isfinite(lse[0, h].cpu().numpy()).all() and torch.isfinite(out[0, :, h].float()).all()
        check_o(out[0, :, h].float().cpu().numpy(), ro, f"growing logits head {h}")
        # LSE values reach a few hundred here: the absolute tolerance is kept, relative to that it is 1e-5
        check_lse(lse[0, h].cpu().numpy(), rl, f"growing logits head {h}")
        for j in range(P):
            so, sl = orc.pair_state(qb, kb, vb, scale, 0, h, rows, int(off[j]), int(off[j + 1]), fp16=fp16)
            check_o(ctx.o_state[j, 0, h].float().cpu().numpy(), so, f"growing logits state {j}")
            check_lse(ctx.lse_state[j, 0, h].cpu().numpy(), sl, f"growing logits state {j}")
    assert lse_max > 150.0      # the case really is extreme


def test_logit_jump_beyond_fp32_range_is_reported():
    """bf16 inputs: the reference of a row moves after the fact by whole binades, which is exact as long as exp2 of a
    logit taken against the previous tiles' reference stays inside fp32.  A logit that rises by more than that within
    one K/V tile (here about 430 binades) cannot be represented: the launch reports DT_ERR_RANGE through dt_poll instead
    of returning a wrong state, and the context stays usable.  fp16 inputs take the tile's own maximum first and have
    no such limit."""
    B, H, D, L, P = 1, 1, 64, 512, 1
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(3)
    u = np.zeros(D, np.float32); u[:4] = 0.5
    q = 0.1 * rng.standard_normal((B, L, H, D)).astype(np.float32) + 10.0 * u
    k = 0.1 * rng.standard_normal((B, L, H, D)).astype(np.float32)
    k[0, 128:, 0, :] += 30.0 * u          # keys of the second tile onwards: logits about 300 (natural units) higher
    v = rng.standard_normal((B, L, H, D)).astype(np.float32)
    off = np.array([0, L], dtype=np.int32)
    mask = torch.ones(P * P, dtype=torch.uint8, device=dev)
    for fp16 in (False, True):
        dt = torch.float16 if fp16 else torch.bfloat16
        qt, kt, vt = (torch.from_numpy(x).to(dt).to(dev) for x in (q, k, v))
        ctx = binding.Context(B, H, D, L, off, 1.0, input_dtype=binding.DT_INPUT_FP16 if fp16 else binding.DT_INPUT_BF16)
        out = torch.empty((B, L, H, D), dtype=dt, device=dev)
        lse = torch.empty((B, H, L), dtype=torch.float32, device=dev)
        ctx.dt_attn_states(qt, kt, vt, mask, 0)
        ctx.dt_state_merge(out, lse)
        if not fp16:
            with pytest.raises(binding.DitangoError) as ei:
                ctx.dt_poll()
            assert ei.value.status == binding.DT_ERR_RANGE
            ctx.dt_poll()                       # the word was cleared: the context is usable again
            kt = torch.from_numpy(k * 0.1).to(dt).to(dev)   # the same shape of inputs with a jump of 43 binades
            ctx.dt_attn_states(qt, kt, vt, mask, 1)
            ctx.dt_state_merge(out, lse)
        ctx.dt_poll()
        qb, kb, vb = (inputs.bf16_bits(x) for x in (qt, kt, vt))
        rows = np.arange(L, dtype=np.int32)
        ro, rl = orc.full_attention(qb, kb, vb, 1.0, 0, 0, rows, fp16=fp16)
        check_o(out[0, :, 0].float().cpu().numpy(), ro, "logit jump")
        check_lse(lse[0, 0].cpu().numpy(), rl, "logit jump")
