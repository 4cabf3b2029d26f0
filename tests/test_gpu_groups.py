"""GPU parity of the grouped state cache (Section 4.2.1, 4.2.2; Eq. 15) through the C ABI against the oracle's
definition (group state = composition of member states).  Same tolerances as the pair-mode tests."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs
from tests.test_gpu_parity import check_lse, check_o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


class GroupRun:
    def __init__(self, wl, g, offsets=None, state_dtype=binding.DT_STATE_FP32, seed=0, rows_by_bh=None, fp16=False):
        self.wl, self.g = wl, g
        self.off = wl.offsets() if offsets is None else np.asarray(offsets, dtype=np.int32)
        self.P = self.off.size - 1
        self.dev = torch.device("cuda", 0)
        in_dt = torch.float16 if fp16 else torch.bfloat16
        self.ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, self.off, wl.scale, state_dtype, 0, group_size=g,
                                   input_dtype=binding.DT_INPUT_FP16 if fp16 else binding.DT_INPUT_BF16)
        self.gen = inputs.StepInputs(wl, seed=seed, device=self.dev, dtype=in_dt)
        if rows_by_bh is None:
            rows_by_bh = {(b, h): np.arange(wl.L, dtype=np.int32) for b in range(wl.B) for h in range(wl.H)}
        self.rows = rows_by_bh
        self.ses = orc.GroupedOracleSession(wl.B, wl.L, wl.H, wl.D, self.off, wl.scale, rows_by_bh, g, fp16=fp16)
        self.out = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=in_dt, device=self.dev)
        self.lse = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=self.dev)
        self.t = 0
        self.tol_scale = 1.0     # raised by tests that compose a bf16 cache in place (see check_o)

    @property
    def S(self):
        return self.ctx.dt_num_slots()[0]

    def check_layout(self):
        S, g = self.ctx.dt_num_slots()
        assert (S, g) == (self.ses.S, self.ses.g)
        rng = self.ctx.dt_slot_ranges()
        for i in range(self.P):
            for s in range(S):
                keys = np.concatenate([np.arange(rng[i, s, 0], rng[i, s, 0] + rng[i, s, 1]),
                                       np.arange(rng[i, s, 2], rng[i, s, 2] + rng[i, s, 3])])
                want = [x for j in self.ses.members[i][s] for x in range(self.off[j], self.off[j + 1])]
                assert keys.tolist() == want, (i, s)

    def check_merged(self, what):
        out_h, lse_h = self.out.float().cpu().numpy(), self.lse.cpu().numpy()
        for (b, h), rows in self.rows.items():
            ro, rl = orc.merge(self.ses.o[(b, h)], self.ses.lse[(b, h)])
            check_o(out_h[b, rows, h, :], ro, f"{what} head {h} merged", self.tol_scale)
            check_lse(lse_h[b, h, rows], rl, f"{what} head {h} merged")

    def check_states(self, what):
        o_st = self.ctx.o_state.float().cpu().numpy()
        l_st = self.ctx.lse_state.cpu().numpy()
        for (b, h), rows in self.rows.items():
            part = np.searchsorted(self.off, rows, side="right") - 1
            for s in range(self.ses.S):
                exists = np.array([bool(self.ses.members[i][s]) for i in part])
                if not exists.any():
                    continue
                check_o(o_st[s, b, h, rows[exists], :], self.ses.o[(b, h)][exists, s, :], f"{what} slot {s}", self.tol_scale)
                check_lse(l_st[s, b, h, rows[exists]], self.ses.lse[(b, h)][exists, s], f"{what} slot {s}")

    def step(self, mask, check_states=True):
        self.t += 1
        q, k, v = self.gen.next()
        mask = np.ascontiguousarray(mask, dtype=np.uint8).reshape(self.P, self.S)
        self.ctx.dt_attn_states(q, k, v, torch.from_numpy(mask).to(self.dev), self.t)
        self.ctx.dt_state_merge(self.out, self.lse)
        torch.cuda.synchronize()
        self.ctx.dt_poll()
        qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
        self.ses.step(qb, kb, vb, mask, self.t)
        self.check_merged(f"step {self.t}")
        if check_states:
            self.check_states(f"step {self.t}")
        tc = self.ctx.dt_get_tc()
        exists = np.array([[bool(self.ses.members[i][s]) for s in range(self.S)] for i in range(self.P)])
        assert (tc[exists] == self.ses.tc[exists]).all()
        return q, k, v


@pytest.mark.parametrize("g", [2, 3, 4])
def test_group_states_config0(g):
    """Correctness config (1024 tokens, P = 4): every slot computed, then only the local slot and one group."""
    wl = inputs.WORKLOADS["c0_correctness"]
    run = GroupRun(wl, g)
    run.check_layout()
    S = run.S
    run.step(np.ones((4, S), np.uint8))
    m = np.zeros((4, S), np.uint8); m[:, 0] = 1; m[:, S - 1] = 1
    run.step(m)
    assert run.ctx.dt_launch_count() == 6


@pytest.mark.parametrize("D,grid,n_text,offsets,g", [
    (128, (4, 11, 13), 0, [0, 129, 385, 572], 2),               # own group with keys on one side only
    (64, (5, 12, 13), 3, [0, 100, 300, 520, 700, 783], 3),       # own group with a hole; last group of two
    (128, (3, 9, 11), 5, [0, 60, 100, 230, 302], 3),             # last group is one partition: no own-group slot for it
    (64, (4, 16, 16), 0, [0, 200, 290, 640, 700, 1024], 5),      # one group: slot 1 = everything but the local keys
])
def test_group_states_ragged(D, grid, n_text, offsets, g):
    wl = inputs.Workload("ragged_groups", 1, 3, D, grid, n_text, len(offsets) - 1, 2, 0.05)
    assert wl.L == offsets[-1]
    P = len(offsets) - 1
    run = GroupRun(wl, g, offsets=offsets, seed=4)
    run.check_layout()
    run.step(np.ones((P, run.S), np.uint8))
    m = np.zeros((P, run.S), np.uint8); m[:, 0] = 1; m[::2, 1] = 1
    run.step(m)


def test_group_states_bf16_cache_and_batch_two():
    wl = inputs.Workload("b2g", 2, 2, 128, (2, 10, 13), 0, 4, 2, 0.05)
    run = GroupRun(wl, 2, state_dtype=binding.DT_STATE_BF16, seed=3)
    run.step(np.ones((4, run.S), np.uint8))
    m = np.zeros((4, run.S), np.uint8); m[:, 0] = 1; m[1, 2] = 1
    run.step(m)


def test_reuse_of_an_empty_slot_is_reported_and_missing_slots_are_not():
    wl = inputs.Workload("empty", 1, 2, 64, (2, 8, 9), 0, 3, 1, 0.05)      # groups {0,1} {2}: partition 2 has no slot 2
    run = GroupRun(wl, 2)
    q, k, v = run.gen.next()
    m = np.zeros((3, run.S), np.uint8); m[:, 0] = 1
    run.ctx.dt_attn_states(q, k, v, torch.from_numpy(m).to(run.dev), 1)
    torch.cuda.synchronize()
    with pytest.raises(binding.DitangoError) as e:
        run.ctx.dt_poll()
    assert e.value.status == binding.DT_ERR_STATE
    full = np.ones((3, run.S), np.uint8); full[2, 2] = 0                   # the slot that does not exist: REUSE is fine
    run.ctx.dt_attn_states(q, k, v, torch.from_numpy(full).to(run.dev), 2)
    run.ctx.dt_attn_states(q, k, v, torch.from_numpy(m).to(run.dev), 3)
    torch.cuda.synchronize()
    run.ctx.dt_poll()


@pytest.mark.parametrize("state_dtype", [binding.DT_STATE_FP32, binding.DT_STATE_BF16])
def test_dynamic_group_compose_in_place(state_dtype):
    """Eq. 15: g = 2 -> 4 -> 8 in place; each composed cache is compared slot by slot with the oracle's
    composition, keeps merging to the same output, and takes further selective steps."""
    wl = inputs.Workload("compose", 1, 2, 64, (4, 12, 13), 0, 8, 3, 0.05)
    run = GroupRun(wl, 2, seed=9, state_dtype=state_dtype)
    run.step(np.ones((8, run.S), np.uint8))
    m = np.zeros((8, run.S), np.uint8); m[:, 0] = 1; m[:, 2] = 1
    run.step(m)
    for expect_S in (3, 2):
        run.ctx.dt_group_compose()
        run.ses.compose()
        run.check_layout()
        assert run.S == expect_S
        torch.cuda.synchronize()
        run.ctx.dt_poll()
        run.check_states(f"composed to S={expect_S}")
        run.ctx.dt_state_merge(run.out, run.lse)
        torch.cuda.synchronize()
        run.check_merged(f"composed to S={expect_S}")
        tc = run.ctx.dt_get_tc()
        assert (tc == run.ses.tc).all()
        m = np.zeros((8, run.S), np.uint8); m[:, 0] = 1; m[3:, 1] = 1
        run.step(m)
    with pytest.raises(binding.DitangoError) as e:
        run.ctx.dt_group_compose()
    assert e.value.status == binding.DT_ERR_STATE
    run.ctx.dt_group_reset()
    run.ses.reset()
    run.check_layout()
    assert (run.ctx.dt_get_tc() == -1).all()
    run.step(np.ones((8, run.S), np.uint8))


def test_slot_plan_matches_oracle_rule():
    """dt_plan on a grouped cache: W per slot against the oracle's slot importance; decisions bit-exact
    against the oracle rule applied to the GPU's own W (threshold and target fraction)."""
    wl = inputs.WORKLOADS["c0_correctness"]
    P = 8
    off = orc.uniform_offsets(wl.L, P)
    run = GroupRun(wl, 2, offsets=off)
    S = run.S
    run.step(np.ones((P, S), np.uint8), check_states=False)
    mem = run.ses.members
    lse_slots = run.ctx.lse_state.double().cpu().numpy()
    W_ref = orc.slot_contribution(lse_slots, off, mem)
    mask_dev = torch.zeros(P * S, dtype=torch.uint8, device=run.dev)
    w_dev = torch.zeros(P * S, dtype=torch.float64, device=run.dev)
    eps_dev = torch.zeros(1, dtype=torch.float64, device=run.dev)
    for kwargs in (dict(eps=0.05), dict(eps=0.2), dict(target_fraction=0.4), dict(target_fraction=0.75),
                   dict(target_fraction=1.0), dict(target_fraction=0.0)):
        run.ctx.dt_plan(mask_dev, w_dev=w_dev, eps_out_dev=eps_dev, **kwargs)
        torch.cuda.synchronize()
        W = w_dev.cpu().numpy().reshape(P, S)
        np.testing.assert_allclose(W, W_ref, rtol=0, atol=2e-6)
        want, eps_want = orc.slot_plan(W, mem, 2, **kwargs)
        assert (mask_dev.cpu().numpy().reshape(P, S) == want).all(), kwargs
        assert eps_dev.item() == pytest.approx(eps_want, abs=1e-15)
    with pytest.raises(binding.DitangoError) as e:
        run.ctx.dt_plan_grouped(mask_dev, 2)
    assert e.value.status == binding.DT_ERR_UNSUPPORTED


def test_composed_reuse_state_on_a_grouped_cache():
    """dt_compose_reuse / dt_state_merge_planned with [P][S] masks."""
    wl = inputs.Workload("planned", 1, 2, 128, (3, 10, 12), 0, 6, 2, 0.05)
    run = GroupRun(wl, 2, seed=6)
    S = run.S
    run.step(np.ones((6, S), np.uint8), check_states=False)
    m = np.zeros((6, S), np.uint8); m[:, 0] = 1; m[:3, 1] = 1; m[4, 3] = 1
    q, k, v = run.step(m, check_states=False)
    mask_dev = torch.from_numpy(m.reshape(-1)).to(run.dev)
    comp_o = torch.empty((wl.B, wl.H, wl.L, wl.D), dtype=torch.float32, device=run.dev)
    comp_l = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32, device=run.dev)
    run.ctx.dt_compose_reuse(mask_dev, comp_o, comp_l)
    out2 = torch.empty_like(run.out); lse2 = torch.empty_like(run.lse)
    run.ctx.dt_state_merge_planned(mask_dev, comp_o, comp_l, out2, lse2)
    torch.cuda.synchronize()
    run.ctx.dt_poll()
    run.out, run.lse = out2, lse2
    run.check_merged("planned merge")


def test_memory_budget_triggers_group_compose():
    """Section 4.2 (Dynamic Group State Compose): compositions run until the slots in use fit the byte budget."""
    wl = inputs.Workload("fit", 1, 2, 64, (4, 12, 13), 0, 8, 2, 0.05)
    run = GroupRun(wl, 2, seed=10)
    run.step(np.ones((8, run.S), np.uint8), check_states=False)
    per_slot = wl.B * wl.H * wl.L * (wl.D * 4 + 4)
    assert run.ctx.dt_group_fit(5 * per_slot) == 0 and run.S == 5          # already fits
    assert run.ctx.dt_group_fit(3 * per_slot + 1) == 1 and run.S == 3      # g 2 -> 4
    run.ses.compose()
    run.check_layout()
    torch.cuda.synchronize()
    run.check_states("fit to 3 slots")
    with pytest.raises(binding.DitangoError) as e:                          # g -> 8 leaves 2 slots: still above 1 slot
        run.ctx.dt_group_fit(per_slot)
    assert e.value.status == binding.DT_ERR_STATE and run.S == 2
    run.ses.compose()
    torch.cuda.synchronize()
    run.check_states("fit to 2 slots")


def test_algorithm1_planner_on_a_grouped_cache_with_a_compose_between_anchors():
    """Algorithm 1 per slot on the device (local attention -> plan -> remaining slots -> merge -> commit) against
    the oracle rule applied to the GPU's own w, alpha and local drift; after step 3 the cache is composed g 2 -> 4
    (Eq. 15) and planning continues on the coarser slots with w and alpha taken again from the composed cache."""
    wl = inputs.Workload("alg1g", 1, 2, 64, (4, 16, 16), 0, 8, 7, 0.05)
    P, R, eps_local = 8, 0.5, 0.5
    run = GroupRun(wl, 2, seed=21)
    dev, ctx, off = run.dev, run.ctx, run.off
    snap_o = torch.zeros((wl.B, wl.H, wl.L, wl.D), dtype=torch.float32, device=dev)
    snap_l = torch.zeros((wl.B, wl.H, wl.L), dtype=torch.float32, device=dev)
    ctx.dt_planner_init(snap_o, snap_l, group_size=1, eps_initial=0.0, eps_local=eps_local, cache_ratio=R)
    with pytest.raises(binding.DitangoError):
        ctx.dt_planner_init(snap_o, snap_l, group_size=2)
    flag = torch.zeros(1, dtype=torch.int32, device=dev)
    drel = torch.zeros(1, dtype=torch.float64, device=dev)
    part = np.searchsorted(off, np.arange(wl.L), side="right") - 1
    eps, have_anchor = 0.0, False
    anchors = selective = 0
    for t in range(wl.steps):
        S = run.S
        mem = run.ses.members
        mask = torch.zeros(P * S, dtype=torch.uint8, device=dev)
        ase = torch.zeros(P * S, dtype=torch.float64, device=dev)
        q, k, v = run.gen.next()
        ctx.dt_attn_local(q, k, v, t)
        ctx.dt_planner_step(mask, flag, ase, drel)
        torch.cuda.synchronize()
        w_g, alpha_g, eps_dev, have_g = ctx.dt_planner_get()
        assert have_g == have_anchor and w_g.shape == (P, S)
        o_c = ctx.o_state[0].double().cpu().numpy(); l_c = ctx.lse_state[0].double().cpu().numpy()   # slot 0: local states
        so = snap_o.double().cpu().numpy(); sl = snap_l.double().cpu().numpy()
        drift = np.zeros(P); base = np.zeros(P)
        for i in range(P):
            rows = part == i
            drift[i] = ((o_c[:, :, rows] - so[:, :, rows]) ** 2).sum() + ((l_c[:, :, rows] - sl[:, :, rows]) ** 2).sum()
            base[i] = (so[:, :, rows] ** 2).sum() + (sl[:, :, rows] ** 2).sum()
        ref = orc.planner_step_slots(w_g, alpha_g, mem, drift, base, eps, eps_local, R, have_anchor)
        got_mask = mask.cpu().numpy().reshape(P, S)
        assert bool(flag.item()) == ref["is_anchor"], (t, ref["delta_rel"])
        assert (got_mask == ref["mask"]).all(), t
        if have_anchor:
            units = ~np.isnan(ref["ase"])
            got_ase = ase.cpu().numpy().reshape(P, S)
            np.testing.assert_allclose(got_ase[units], ref["ase"][units], rtol=1e-4)
            assert np.isnan(got_ase[~units]).all()
            assert drel.item() == pytest.approx(ref["delta_rel"], rel=1e-4)
            if not ref["is_anchor"]:
                assert (np.abs(ref["ase"][units] - eps) / max(eps, 1e-300)).min() > 1e-5
        assert eps_dev == pytest.approx(ref["eps"], rel=1e-4)
        eps = eps_dev
        rest = got_mask.copy(); rest[:, 0] = 0
        ctx.dt_attn_states(q, k, v, torch.from_numpy(rest.reshape(-1).copy()).to(dev), t)
        ctx.dt_state_merge(run.out, run.lse)
        ctx.dt_planner_commit()
        torch.cuda.synchronize()
        ctx.dt_poll()
        run.ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), got_mask, t)
        run.check_merged(f"alg1 grouped step {t}")
        assert (ctx.dt_get_tc() == run.ses.tc).all()

        def check_stats(what):
            """w (Eq. 8 / Eq. 12) and alpha (Eq. 9) against the oracle's states."""
            w_g, alpha_g, _, _ = ctx.dt_planner_get()
            S = run.ses.S
            lse_ref = np.empty((S, wl.B, wl.H, wl.L)); nsq = np.zeros((P, S))
            for (b, h), _rows in run.rows.items():
                lse_ref[:, b, h, :] = run.ses.lse[(b, h)].T
                for i in range(P):
                    sel = part == i
                    for s in range(S):
                        if run.ses.members[i][s]:
                            nsq[i, s] += orc.state_norm_sq(run.ses.o[(b, h)][sel, s, :], run.ses.lse[(b, h)][sel, s])
            np.testing.assert_allclose(w_g, orc.slot_contribution(lse_ref, off, run.ses.members), rtol=2e-3, atol=1e-6, err_msg=what)
            np.testing.assert_allclose(alpha_g, np.sqrt(nsq / nsq[:, :1]), rtol=2e-3, err_msg=what)

        if ref["is_anchor"]:
            anchors += 1
            have_anchor = True
            check_stats(f"anchor at step {t}")
            assert torch.equal(snap_l, ctx.lse_state[0])
        else:
            selective += 1
            assert P <= got_mask.sum() < P * S
        if t == 3:
            ctx.dt_group_compose()
            run.ses.compose()
            torch.cuda.synchronize()
            assert run.S == 3
            check_stats("after compose")
    assert anchors >= 2 and selective >= 2
