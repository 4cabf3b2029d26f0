"""Pins for the grouped-cache part of the oracle (Section 4.2.1, 4.2.2; Eq. 15): group states are defined
by composition (Eq. 2) of member states; these tests tie that definition to quantities computed another way."""
import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import oracle as orc
from tests.test_oracle_pins import all_rows, rand_qkv, widen


def test_group_slots_structure():
    """Section 4.2.1: p/g groups of g states; the group holding the local state has g - 1."""
    mem = orc.group_slots(8, 4)
    assert len(mem[0]) == 3                                  # local + 2 groups
    assert mem[5][0] == [5] and mem[5][1] == [0, 1, 2, 3] and mem[5][2] == [4, 6, 7]
    mem = orc.group_slots(7, 3)                              # groups {0,1,2} {3,4,5} {6}
    assert mem[6][3] == [] and mem[6][1] == [0, 1, 2] and mem[0][1] == [1, 2] and mem[0][3] == [6]
    for i in range(7):                                       # every KV partition appears exactly once per query partition
        flat = sorted(j for s in mem[i] for j in s)
        assert flat == list(range(7))
    mem1 = orc.group_slots(4, 1)                             # g = 1: one partition per group, the own group is empty
    assert mem1[2] == [[2], [0], [1], [], [3]]


def _brute_state(q, k, v, scale, b, h, row, keys):
    """Eq. 1 written with numpy for an arbitrary key set."""
    Q, K, V = widen(q)[b, row, h], widen(k)[b, keys, h], widen(v)[b, keys, h]
    x = scale * (K @ Q)
    m = x.max()
    e = np.exp(x - m)
    return (e[:, None] * V).sum(0) / e.sum(), m + np.log(e.sum())


@pytest.mark.parametrize("P,g,off", [(6, 2, None), (7, 3, None), (5, 4, (0, 5, 9, 20, 26, 33))])
def test_group_state_by_composition_equals_one_softmax_over_the_groups_keys(P, g, off):
    """Eq. 2 / Eq. 15: composing the member states of a group gives the state over the union of their keys,
    also for the own group, whose keys lie on both sides of the local partition."""
    rng = np.random.default_rng(5)
    L = 33
    off = orc.uniform_offsets(L, P) if off is None else np.array(off, dtype=np.int32)
    q, k, v = rand_qkv(rng, 1, L, 2, 8, 1.3)
    rows = {(0, 1): all_rows(L)}
    ses = orc.GroupedOracleSession(1, L, 2, 8, off, 0.4, rows, g)
    mask = np.ones((P, ses.S), dtype=np.uint8)
    outs, lses = ses.step(q, k, v, mask, 0)
    part = np.searchsorted(off, all_rows(L), side="right") - 1
    for r in range(L):
        i = part[r]
        for s in range(ses.S):
            mem = ses.members[i][s]
            if not mem:
                assert ses.lse[(0, 1)][r, s] == -np.inf
                continue
            keys = np.concatenate([np.arange(off[j], off[j + 1]) for j in mem])
            o, l = _brute_state(q, k, v, 0.4, 0, 1, r, keys)
            np.testing.assert_allclose(ses.o[(0, 1)][r, s], o, rtol=0, atol=1e-12)
            np.testing.assert_allclose(ses.lse[(0, 1)][r, s], l, rtol=0, atol=1e-12)
    # a remote group is contiguous: the C routine over [off[lo], off[hi]) must agree as well
    o, l = orc.pair_state(q, k, v, 0.4, 0, 1, all_rows(off[1]), int(off[g]), int(off[min(P, 2 * g)]))
    np.testing.assert_allclose(ses.o[(0, 1)][:off[1], 2], o, rtol=0, atol=1e-12)
    # all slots together are full attention
    fo, fl = orc.full_attention(q, k, v, 0.4, 0, 1, all_rows(L))
    np.testing.assert_allclose(outs[(0, 1)], fo, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lses[(0, 1)], fl, rtol=0, atol=1e-12)


def test_dynamic_group_compose_gives_the_states_of_the_coarser_grouping():
    """Eq. 15 with k = 2: composing adjacent group states g -> 2g equals computing with 2g directly; the
    composed cache still merges to full attention; t_c of a composed slot is the older of its sources."""
    rng = np.random.default_rng(6)
    P, L, g = 8, 41, 2
    off = orc.uniform_offsets(L, P)
    q, k, v = rand_qkv(rng, 1, L, 1, 8, 1.1)
    rows = {(0, 0): all_rows(L)}
    a = orc.GroupedOracleSession(1, L, 1, 8, off, 0.5, rows, g)
    b = orc.GroupedOracleSession(1, L, 1, 8, off, 0.5, rows, 2 * g)
    a.step(q, k, v, np.ones((P, a.S), dtype=np.uint8), 0)
    m1 = np.zeros((P, a.S), dtype=np.uint8); m1[:, 0] = 1; m1[:, 1] = 1          # step 1 recomputes group 0 only
    a.step(q, k, v, m1, 1)
    outs_b, _ = b.step(q, k, v, np.ones((P, b.S), dtype=np.uint8), 0)
    a.compose()
    assert a.S == b.S == 3 and a.g == 4
    np.testing.assert_allclose(a.o[(0, 0)], b.o[(0, 0)], rtol=0, atol=1e-12)
    np.testing.assert_allclose(a.lse[(0, 0)], b.lse[(0, 0)], rtol=0, atol=1e-12)
    o, l = orc.merge(a.o[(0, 0)], a.lse[(0, 0)])
    np.testing.assert_allclose(o, outs_b[(0, 0)], rtol=0, atol=1e-12)
    # new slot 1 = old slots 1 (t_c 1) and 2 (t_c 0) -> 0; new slot 2 = old 3, 4 -> 0; partitions 0, 1: old slot 1 is
    # their own group, which exists for both (one other member)
    assert (a.tc[:, 0] == 1).all() and (a.tc[:, 1] == 0).all() and (a.tc[:, 2] == 0).all()
    a.compose()
    assert a.S == 2 and a.g == 8
    a.reset()
    assert a.S == 5 and (a.tc == -1).all()


def test_slot_importance_is_the_sum_of_member_importances():
    """Eq. 12: a group's measure is the sum over its members; from the group's LSE this is exp(LSE_G - LSE)."""
    rng = np.random.default_rng(7)
    P, g, B, H, L = 6, 2, 1, 2, 30
    off = orc.uniform_offsets(L, P)
    lse_pair = rng.standard_normal((P, B, H, L)) * 2.0
    W = orc.contribution(lse_pair, off)
    mem = orc.group_slots(P, g)
    S = len(mem[0])
    lse_slot = np.full((S, B, H, L), -np.inf)
    for i in range(P):
        for s in range(S):
            if mem[i][s]:
                x = lse_pair[mem[i][s]][:, :, :, off[i]:off[i + 1]]
                lse_slot[s, :, :, off[i]:off[i + 1]] = np.log(np.exp(x).sum(axis=0))
    Ws = orc.slot_contribution(lse_slot, off, mem)
    for i in range(P):
        for s in range(S):
            np.testing.assert_allclose(Ws[i, s], sum(W[i, j] for j in mem[i][s]), rtol=0, atol=1e-12)
    np.testing.assert_allclose(Ws.sum(axis=1), 1.0, atol=1e-12)
    # closed form against a library softmax for one row-partition
    x = lse_slot[:, 0, 0, off[2]:off[3]]
    np.testing.assert_allclose(orc.slot_contribution(lse_slot[:, :1, :1], off, mem)[2],
                               sp_softmax(x, axis=0).mean(axis=1), atol=1e-12)


@pytest.mark.parametrize("P,g", [(8, 2), (8, 4), (6, 3)])
def test_slot_plan_agrees_with_the_group_rule_on_pairs(P, g):
    """The per-slot rule must take the same decisions as the pair-level group rule (orc_group_plan): the
    same units with the same measures, thresholded or ranked the same way."""
    rng = np.random.default_rng(8 + P + g)
    W = rng.random((P, P)) ** 3
    W /= W.sum(axis=1, keepdims=True)
    mem = orc.group_slots(P, g)
    S = len(mem[0])
    Ws = np.array([[sum(W[i, j] for j in mem[i][s]) for s in range(S)] for i in range(P)])
    for kwargs in (dict(eps=0.12), dict(eps=0.0), dict(target_fraction=0.4), dict(target_fraction=0.7),
                   dict(target_fraction=1.0), dict(target_fraction=0.0)):
        mp, eps_p, _ = orc.group_plan(W, g, **kwargs)
        ms, eps_s = orc.slot_plan(Ws, mem, g, **kwargs)
        assert (ms[:, 0] == 1).all()
        for i in range(P):
            for s in range(1, S):
                for j in mem[i][s]:
                    assert ms[i, s] == mp[i, j], (kwargs, i, s, j)
        assert eps_s == pytest.approx(eps_p, abs=1e-15)
    # strict inequality: a slot exactly at eps is reused
    ms, _ = orc.slot_plan(Ws, mem, g, eps=float(Ws[0, 1]))
    assert ms[0, 1] == 0


def test_planner_rule_on_slots_reduces_to_the_pair_rule_when_every_group_is_one_partition():
    """Algorithm 1 per slot: with groups of one partition the units, their ASE (Eq. 7, 10, 12), the anchor test
    (Eq. 14), the threshold (Eq. 13) and the eps update must be those of the pair-level rule."""
    rng = np.random.default_rng(11)
    P = 5
    mem = orc.group_slots(P, 1)                      # slot 0 local, slot 1 + j = [j] (empty for j == i)
    S = P + 1
    W = rng.random((P, P)); W /= W.sum(axis=1, keepdims=True)
    alpha = 0.5 + rng.random((P, P)); alpha[np.arange(P), np.arange(P)] = 1.0
    Ws = np.zeros((P, S)); As = np.zeros((P, S))
    for i in range(P):
        Ws[i, 0], As[i, 0] = W[i, i], 1.0
        for j in range(P):
            if j != i:
                Ws[i, 1 + j], As[i, 1 + j] = W[i, j], alpha[i, j]
    base = 1.0 + rng.random(P)
    for scale, eps, have in ((1e-3, 0.02, True), (0.2, 0.02, True), (0.05, 0.004, True), (0.05, 0.02, False),
                             (0.0, 0.0, True), (3.0, 0.02, True)):
        drift = scale * rng.random(P)
        a = orc.planner_step(W, alpha, drift, base, 1, eps, 0.4, 0.6, have)
        b = orc.planner_step_slots(Ws, As, mem, drift, base, eps, 0.4, 0.6, have)
        assert a["is_anchor"] == b["is_anchor"] and a["eps"] == pytest.approx(b["eps"], rel=1e-15)
        assert a["delta_rel"] == b["delta_rel"]
        for i in range(P):
            assert b["mask"][i, 0] == 1
            for j in range(P):
                if j != i:
                    assert a["mask"][i, j] == b["mask"][i, 1 + j]
                    assert a["ase"][i, j] == pytest.approx(b["ase"][i, 1 + j], rel=1e-15)
