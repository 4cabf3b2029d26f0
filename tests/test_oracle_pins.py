"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix, never the oracle itself.

Each test names the passage it pins.  A dropped term, wrong sign, swapped index or
transposed operand in oracle/ditango_oracle.c should fail at least one of these.
"""
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import logsumexp as sp_logsumexp
from scipy.special import softmax as sp_softmax

from oracle import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def widen(bits: np.ndarray) -> np.ndarray:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()


def rand_qkv(rng, B, L, H, D, spread=1.0):
    return tuple(bf16_bits(rng.standard_normal((B, L, H, D)) * spread) for _ in range(3))


def all_rows(L):
    return np.arange(L, dtype=np.int32)


# ---------------------------------------------------------------- Eq. 1 and full attention

def test_full_attention_matches_library_sdpa():
    """softmax(s QK^T)V (the definition Eq. 1 + Eq. 2 must reproduce) against torch's fp64 SDPA
    and scipy's logsumexp."""
    rng = np.random.default_rng(1)
    B, L, H, D = 2, 37, 3, 16
    q, k, v = rand_qkv(rng, B, L, H, D, 1.5)
    s = 0.37
    qt, kt, vt = (torch.from_numpy(widen(x)).permute(0, 2, 1, 3) for x in (q, k, v))     # [B,H,L,D]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=s).numpy()
    logits = s * torch.matmul(qt, kt.transpose(-1, -2)).numpy()
    ref_lse = sp_logsumexp(logits, axis=-1)
    for b in range(B):
        for h in range(H):
            o, lse = orc.full_attention(q, k, v, s, b, h, all_rows(L))
            np.testing.assert_allclose(o, ref[b, h], rtol=0, atol=1e-13)
            np.testing.assert_allclose(lse, ref_lse[b, h], rtol=0, atol=1e-13)


def test_two_key_hand_example():
    """Eq. 1 by hand: q = e0, k1 = e0, k2 = 0  ->  x = (s, 0), LSE = log(e^s + 1),
    OUT = (e^s v1 + v2) / (e^s + 1).  All values exactly representable in bf16."""
    D, s = 8, 0.5
    q = np.zeros((1, 2, 1, D)); k = np.zeros((1, 2, 1, D)); v = np.zeros((1, 2, 1, D))
    q[0, 0, 0, 0] = 1.0
    q[0, 1, 0, 1] = 2.0
    k[0, 0, 0, 0] = 1.0
    v[0, 0, 0, :] = np.arange(D)
    v[0, 1, 0, :] = -2.0
    qb, kb, vb = bf16_bits(q), bf16_bits(k), bf16_bits(v)
    o, lse = orc.pair_state(qb, kb, vb, s, 0, 0, [0, 1], 0, 2)
    e = math.exp(s)
    assert lse[0] == pytest.approx(math.log(e + 1.0), abs=1e-15)
    np.testing.assert_allclose(o[0], (e * np.arange(D) - 2.0) / (e + 1.0), atol=1e-15)
    # row 1 is orthogonal to both keys: uniform weights
    assert lse[1] == pytest.approx(math.log(2.0), abs=1e-15)
    np.testing.assert_allclose(o[1], (np.arange(D) - 2.0) / 2.0, atol=1e-15)
    # a single-key partition returns that key's value and its logit
    o1, l1 = orc.pair_state(qb, kb, vb, s, 0, 0, [0], 0, 1)
    np.testing.assert_allclose(o1[0], np.arange(D), atol=0)
    assert l1[0] == pytest.approx(s, abs=1e-15)


def test_zero_keys_closed_form():
    """K == 0: every logit is 0, so LSE_ij = ln n_j and OUT_ij = mean of V over partition j."""
    rng = np.random.default_rng(2)
    B, L, H, D = 1, 29, 2, 8
    q, _, v = rand_qkv(rng, B, L, H, D)
    k = np.zeros_like(q)
    off = [0, 5, 18, 29]
    vw = widen(v)
    for j in range(3):
        o, lse = orc.pair_state(q, k, v, 0.3, 0, 1, all_rows(L), off[j], off[j + 1])
        np.testing.assert_allclose(lse, math.log(off[j + 1] - off[j]), atol=1e-14)
        mean_v = vw[0, off[j]:off[j + 1], 1, :].mean(axis=0)
        np.testing.assert_allclose(o, np.broadcast_to(mean_v, o.shape), atol=1e-14)


def test_key_permutation_invariance_and_value_hull():
    """A partition's state does not depend on the order of its keys, and OUT_ij is a convex
    combination of the partition's value rows (Eq. 1 weights are positive and sum to 1)."""
    rng = np.random.default_rng(3)
    B, L, H, D = 1, 40, 2, 8
    q, k, v = rand_qkv(rng, B, L, H, D, 2.0)
    lo, hi = 11, 33
    perm = np.arange(L)
    perm[lo:hi] = lo + rng.permutation(hi - lo)
    k2, v2 = k[:, perm].copy(), v[:, perm].copy()
    o, lse = orc.pair_state(q, k, v, 0.5, 0, 0, all_rows(L), lo, hi)
    o2, lse2 = orc.pair_state(q, k2, v2, 0.5, 0, 0, all_rows(L), lo, hi)
    np.testing.assert_allclose(o, o2, atol=1e-13)
    np.testing.assert_allclose(lse, lse2, atol=1e-13)
    vw = widen(v)[0, lo:hi, 0, :]
    assert (o <= vw.max(axis=0) + 1e-14).all() and (o >= vw.min(axis=0) - 1e-14).all()


@pytest.mark.parametrize("offsets", [[0, 31], [0, 16, 31], [0, 3, 4, 20, 31], list(range(32))])
def test_composing_all_partitions_reproduces_full_attention(offsets):
    """Composability (Eq. 2) + completeness: merging the states of all partitions equals plain
    full attention, for any contiguous partitioning (even, uneven, single-key)."""
    rng = np.random.default_rng(4)
    B, L, H, D = 1, 31, 2, 16
    q, k, v = rand_qkv(rng, B, L, H, D, 2.0)
    s = 1.0 / math.sqrt(D)
    P = len(offsets) - 1
    for h in range(H):
        os_ = np.empty((L, P, D)); ls_ = np.empty((L, P))
        for j in range(P):
            os_[:, j], ls_[:, j] = orc.pair_state(q, k, v, s, 0, h, all_rows(L), offsets[j], offsets[j + 1])
        o, lse = orc.merge(os_, ls_)
        fo, flse = orc.full_attention(q, k, v, s, 0, h, all_rows(L))
        np.testing.assert_allclose(o, fo, atol=1e-12)
        np.testing.assert_allclose(lse, flse, atol=1e-12)


# ---------------------------------------------------------------- Eq. 2 algebra

def _random_states(rng, P, D, spread=3.0):
    return rng.standard_normal((P, D)), rng.standard_normal(P) * spread


def test_compose_two_states_matches_eq2_written_with_library_calls():
    """Eq. 2 evaluated with numpy's exp/log directly on moderate LSE values."""
    rng = np.random.default_rng(5)
    o, l = _random_states(rng, 2, 6, 1.0)
    got_o, got_l = orc.compose2(o[0], l[0], o[1], l[1])
    ea, eb = np.exp(l[0]), np.exp(l[1])
    np.testing.assert_allclose(got_o, (ea * o[0] + eb * o[1]) / (ea + eb), atol=1e-14)
    assert got_l == pytest.approx(np.log(ea + eb), abs=1e-14)
    # large LSEs must not overflow (e^800 is not representable)
    big_o, big_l = orc.compose2(o[0], 800.0, o[1], 801.0)
    w = 1.0 / (1.0 + math.e)
    np.testing.assert_allclose(big_o, w * o[0] + (1 - w) * o[1], atol=1e-14)
    assert big_l == pytest.approx(801.0 + math.log1p(math.exp(-1.0)), abs=1e-12)


def test_compose_is_commutative_and_associative_and_matches_fold():
    """(+) is associative and commutative: random orders and random binary trees agree with the
    one-pass P-way merge."""
    rng = np.random.default_rng(6)
    P, D = 7, 5
    o, l = _random_states(rng, P, D)
    ref_o, ref_l = orc.merge(o[None], l[None])

    def tree(items):
        if len(items) == 1:
            return items[0]
        cut = rng.integers(1, len(items))
        a, b = tree(items[:cut]), tree(items[cut:])
        return orc.compose2(a[0], a[1], b[0], b[1])

    for _ in range(20):
        order = rng.permutation(P)
        got_o, got_l = tree([(o[j], l[j]) for j in order])
        np.testing.assert_allclose(got_o, ref_o[0], atol=1e-12)
        assert got_l == pytest.approx(ref_l[0], abs=1e-12)
    ab = orc.compose2(o[0], l[0], o[1], l[1])
    ba = orc.compose2(o[1], l[1], o[0], l[0])
    np.testing.assert_allclose(ab[0], ba[0], atol=0)
    assert ab[1] == ba[1]


def test_first_order_error_propagation_identity():
    """Eq. 3-4: dOUT = w1 dO1 + w2 dO2 + w1 w2 (O1 - O2)(dLSE1 - dLSE2), dLSE = w1 dLSE1 + w2 dLSE2,
    with w_i = e^{LSE_i} / (e^{LSE_1} + e^{LSE_2}).  Checked by finite differences of the
    oracle's compose: the residual must be second order (quarter when the step halves)."""
    rng = np.random.default_rng(7)
    D = 6
    o, l = _random_states(rng, 2, D, 1.0)
    do, dl = rng.standard_normal((2, D)), rng.standard_normal(2)
    base_o, base_l = orc.compose2(o[0], l[0], o[1], l[1])
    w1 = math.exp(l[0]) / (math.exp(l[0]) + math.exp(l[1]))
    w2 = 1.0 - w1
    lin_o = w1 * do[0] + w2 * do[1] + w1 * w2 * (o[0] - o[1]) * (dl[0] - dl[1])
    lin_l = w1 * dl[0] + w2 * dl[1]
    res = []
    for eps in (1e-3, 5e-4):
        po, pl = orc.compose2(o[0] + eps * do[0], l[0] + eps * dl[0], o[1] + eps * do[1], l[1] + eps * dl[1])
        r_o = np.abs(po - base_o - eps * lin_o).max()
        r_l = abs(pl - base_l - eps * lin_l)
        res.append((r_o, r_l))
        assert r_o < 5.0 * eps * eps and r_l < 5.0 * eps * eps
    assert res[1][0] == pytest.approx(res[0][0] / 4.0, rel=0.05)
    assert res[1][1] == pytest.approx(res[0][1] / 4.0, rel=0.05)


def _structural_examples():
    out = []
    with open(os.path.join(GOLDEN, "structural_examples.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, p, computed, reused = [x.strip() for x in line.split("|")]
            out.append((name, int(p), [int(x) for x in computed.split()], [int(x) for x in reused.split()]))
    return out


@pytest.mark.parametrize("name,P,computed,reused", _structural_examples())
def test_precomposed_reuse_states_merge_like_individual_ones(name, P, computed, reused):
    """Fig. 6 (CP = 4, rank 0: compute {0, 1}, reuse the cached composition 2 (+) 3) and the
    8-partition example of Section 5.2: composing the reused states first and then merging with
    the computed ones equals merging all P states."""
    assert sorted(computed + reused) == list(range(P))
    rng = np.random.default_rng(8)
    D = 4
    o, l = _random_states(rng, P, D)
    ref_o, ref_l = orc.merge(o[None], l[None])
    acc = (o[reused[0]], l[reused[0]])
    for j in reused[1:]:
        acc = orc.compose2(acc[0], acc[1], o[j], l[j])
    so = np.stack([o[j] for j in computed] + [acc[0]])
    sl = np.array([l[j] for j in computed] + [acc[1]])
    got_o, got_l = orc.merge(so[None], sl[None])
    np.testing.assert_allclose(got_o, ref_o, atol=1e-13)
    np.testing.assert_allclose(got_l, ref_l, atol=1e-13)


def test_minus_infinity_state_has_zero_weight():
    o = np.ones((1, 3, 2)); o[0, 1] = 7.0
    l = np.array([[0.0, -np.inf, 0.0]])
    got_o, got_l = orc.merge(o, l)
    np.testing.assert_allclose(got_o, 1.0)
    assert got_l[0] == pytest.approx(math.log(2.0))
    z_o, z_l = orc.merge(o, np.full((1, 3), -np.inf))
    assert (z_o == 0).all() and z_l[0] == -np.inf


# ---------------------------------------------------------------- step semantics

def _session(rng, B=1, L=24, H=2, D=8, off=(0, 7, 13, 24)):
    q, k, v = rand_qkv(rng, B, L, H, D, 1.5)
    rows = {(0, h): all_rows(L) for h in range(H)}
    return orc.OracleSession(B, L, H, D, off, 0.4, rows), (q, k, v)


def test_reusing_states_of_identical_inputs_is_exact():
    """Reuse error comes only from AS_t - AS_tc: with unchanged inputs, a banded plan at step 2
    reproduces full attention exactly."""
    rng = np.random.default_rng(9)
    ses, (q, k, v) = _session(rng)
    P = ses.P
    ses.step(q, k, v, np.ones((P, P), np.uint8), 1)
    band = (np.abs(np.subtract.outer(np.arange(P), np.arange(P))) <= 0).astype(np.uint8)
    outs, lses = ses.step(q, k, v, band, 2)
    for (b, h), o in outs.items():
        fo, fl = orc.full_attention(q, k, v, 0.4, b, h, all_rows(24))
        np.testing.assert_allclose(o, fo, atol=1e-12)
        np.testing.assert_allclose(lses[(b, h)], fl, atol=1e-12)
    assert (ses.tc.diagonal() == 2).all() and ses.tc[0, 1] == 1


def test_all_compute_every_step_equals_full_attention_and_reuse_is_stale():
    rng = np.random.default_rng(10)
    ses, (q, k, v) = _session(rng)
    P = ses.P
    q2, k2, v2 = rand_qkv(rng, 1, 24, 2, 8, 1.5)
    ones = np.ones((P, P), np.uint8)
    ses.step(q, k, v, ones, 1)
    outs, _ = ses.step(q2, k2, v2, ones, 2)
    fo, _ = orc.full_attention(q2, k2, v2, 0.4, 0, 1, all_rows(24))
    np.testing.assert_allclose(outs[(0, 1)], fo, atol=1e-12)
    # now reuse pair (0, 2) from step 2 while inputs go back to step 1's: rows of partition 0
    # must equal compose(fresh(0,0), fresh(0,1), stale(0,2)), and differ from full attention
    mask = ones.copy(); mask[0, 2] = 0
    outs3, _ = ses.step(q, k, v, mask, 3)
    rows0 = np.arange(0, 7, dtype=np.int32)
    st = [orc.pair_state(q, k, v, 0.4, 0, 0, rows0, 0, 7), orc.pair_state(q, k, v, 0.4, 0, 0, rows0, 7, 13),
          orc.pair_state(q2, k2, v2, 0.4, 0, 0, rows0, 13, 24)]
    exp_o, _ = orc.merge(np.stack([s[0] for s in st], 1), np.stack([s[1] for s in st], 1))
    np.testing.assert_allclose(outs3[(0, 0)][:7], exp_o, atol=1e-13)
    fo1, _ = orc.full_attention(q, k, v, 0.4, 0, 0, all_rows(24))
    assert np.abs(outs3[(0, 0)][:7] - fo1[:7]).max() > 1e-3
    np.testing.assert_allclose(outs3[(0, 0)][7:], fo1[7:], atol=1e-12)
    assert ses.tc[0, 2] == 2 and ses.tc[0, 0] == 3


def test_reuse_before_compute_is_an_error():
    rng = np.random.default_rng(11)
    ses, (q, k, v) = _session(rng)
    with pytest.raises(RuntimeError):
        ses.step(q, k, v, np.eye(ses.P, dtype=np.uint8), 1)


# ---------------------------------------------------------------- Eq. 8 contribution, Eq. 13 threshold

def test_contribution_rows_sum_to_one_and_match_library_softmax():
    """w is a softmax over partitions (Eq. 8): each row of W sums to 1, and W equals the mean of
    scipy's softmax over the partition axis."""
    rng = np.random.default_rng(12)
    P, B, H, L = 5, 2, 3, 23
    off = np.array([0, 4, 9, 10, 17, 23], np.int32)
    lse = rng.standard_normal((P, B, H, L)) * 2.0
    W = orc.contribution(lse, off)
    np.testing.assert_allclose(W.sum(axis=1), 1.0, atol=1e-14)
    sm = sp_softmax(lse, axis=0)
    for i in range(P):
        np.testing.assert_allclose(W[i], sm[:, :, :, off[i]:off[i + 1]].mean(axis=(1, 2, 3)), atol=1e-14)


def test_contribution_zero_keys_closed_form():
    """K == 0 gives LSE_ij = ln n_j, so W[i][j] = n_j / L for uneven partitions."""
    rng = np.random.default_rng(13)
    B, L, H, D = 1, 26, 2, 8
    off = np.array([0, 3, 11, 26], np.int32)
    q, _, v = rand_qkv(rng, B, L, H, D)
    k = np.zeros_like(q)
    lse = np.empty((3, B, H, L))
    for j in range(3):
        for h in range(H):
            lse[j, 0, h] = orc.pair_state(q, k, v, 0.2, 0, h, all_rows(L), off[j], off[j + 1])[1]
    W = orc.contribution(lse, off)
    n = np.diff(off) / L
    np.testing.assert_allclose(W, np.broadcast_to(n, (3, 3)), atol=1e-14)


def test_contribution_distance_decay_closed_form():
    """Synthetic LSE_ij = -c |i - j| (constant over rows): W[i][j] = e^{-c|i-j|} / sum_k e^{-c|i-k|}."""
    P, B, H, L, c = 6, 1, 2, 18, 0.7
    off = orc.uniform_offsets(L, P)
    lse = np.empty((P, B, H, L))
    for i in range(P):
        for j in range(P):
            lse[j, :, :, off[i]:off[i + 1]] = -c * abs(i - j)
    W = orc.contribution(lse, off)
    for i in range(P):
        e = np.exp(-c * np.abs(np.arange(P) - i))
        np.testing.assert_allclose(W[i], e / e.sum(), atol=1e-15)


def test_threshold_is_strict_and_diagonal_is_always_computed():
    """Eq. 13: COMPUTE iff measure > eps (equality -> REUSE); the local partition is always computed."""
    W = np.array([[0.0, 0.25, 0.5], [0.25, 0.1, 0.2500000001], [0.9, 0.0, 0.0]])
    m = orc.threshold(W, 0.25)
    assert m.tolist() == [[1, 0, 1], [0, 1, 1], [1, 0, 1]]
    assert orc.threshold(W, 10.0).tolist() == np.eye(3, dtype=int).tolist()
    assert orc.threshold(W, -1.0).sum() == 9


def test_target_fraction_invariants():
    rng = np.random.default_rng(14)
    P = 8
    W = rng.random((P, P)); W /= W.sum(1, keepdims=True)
    prev = None
    for f in (0.0, 1.0 / P, 0.2, 0.4, 0.5, 0.77, 1.0):
        mask, eps, K = orc.target_fraction(W, f)
        assert K == min(max(int(math.floor(f * P * P + 0.5)), P), P * P)
        assert mask.sum() == K and (mask.diagonal() == 1).all()
        # the selection is exactly "W > eps" off the diagonal (no ties in random data)
        assert (orc.threshold(W, eps) == mask).all()
        offd = ~np.eye(P, dtype=bool)
        if 0 < (mask[offd] == 0).sum() and (mask[offd] == 1).sum() > 0:
            assert W[offd & (mask == 1)].min() > eps > W[offd & (mask == 0)].max()
        if prev is not None:
            assert (mask >= prev).all()          # nested as f grows
        prev = mask
    assert orc.target_fraction(W, 1.0)[0].all()
    assert (orc.target_fraction(W, 1.0 / P)[0] == np.eye(P)).all()


def test_target_fraction_banded_measure_gives_banded_mask_and_tie_rule():
    """A measure that depends only on |i - j| and decays selects whole diagonals in order; at a tie
    the pair with smaller i*P+j goes first."""
    P = 6
    d = np.abs(np.subtract.outer(np.arange(P), np.arange(P)))
    W = np.exp(-1.3 * d)
    mask, eps, K = orc.target_fraction(W, (P + 2 * (P - 1)) / (P * P))
    assert (mask == (d <= 1)).all() and K == P + 2 * (P - 1)
    assert math.exp(-2.6) < eps < math.exp(-1.3)
    mask1, _, _ = orc.target_fraction(W, (P + 1) / (P * P))
    assert mask1.sum() == P + 1 and mask1[0, 1] == 1


def test_target_fraction_ties_go_to_the_nearer_partition_and_eps_is_the_midpoint():
    """Hand-checked: a measure with only two values, so that the rank order is decided by the tie rule alone --
    equal W: the pair with the smaller |i - j| first, then the smaller i*P + j -- and the reported threshold is the
    midpoint between the last selected and the first unselected value."""
    P = 4
    W = np.full((P, P), 0.1)
    W[0, 3] = W[3, 0] = 0.3                       # the two far corners carry the large value
    # K = 4 + 2: the two corners (largest W) and nothing else; eps midway between 0.3 and 0.1
    mask, eps, K = orc.target_fraction(W, 6 / 16)
    want = np.eye(P, dtype=np.uint8); want[0, 3] = want[3, 0] = 1
    assert K == 6 and (mask == want).all() and eps == 0.5 * (0.3 + 0.1)
    # K = 4 + 2 + 3: among the ten tied pairs the distance-1 ones come first, in index order: (0,1), (1,0), (1,2)
    mask, eps, K = orc.target_fraction(W, 9 / 16)
    want[0, 1] = want[1, 0] = want[1, 2] = 1
    assert K == 9 and (mask == want).all() and eps == 0.1        # the cut runs through a tie: eps is the tied value
    # K = 4 + 2 + 6 + 1: all six distance-1 pairs, then the first distance-2 pair (0,2); (2,0) and the rest stay REUSE
    mask, eps, K = orc.target_fraction(W, 13 / 16)
    d = np.abs(np.subtract.outer(np.arange(P), np.arange(P)))
    want = ((d <= 1) | (d == 3)).astype(np.uint8); want[0, 2] = 1
    assert K == 13 and (mask == want).all()
    # a tie across distances with the larger value on the far pair: value wins over distance
    W2 = np.full((P, P), 0.2); W2[0, 2] = 0.25
    mask, eps, K = orc.target_fraction(W2, 5 / 16)
    assert K == 5 and mask[0, 2] == 1 and mask.sum() == 5 and eps == 0.5 * (0.25 + 0.2)


def test_group_plan_with_group_size_one_is_the_ungrouped_rule():
    """g = 1: every unit is a single off-diagonal pair, so the grouped rule must reproduce Eq. 13 and
    the target-fraction selection exactly."""
    rng = np.random.default_rng(15)
    P = 7
    W = rng.random((P, P)); W /= W.sum(1, keepdims=True)
    for eps in (0.05, 0.12, 0.3):
        m, e, n = orc.group_plan(W, 1, eps=eps)
        assert (m == orc.threshold(W, eps)).all() and e == eps and n == m.sum()
    for f in (0.0, 0.3, 0.5, 0.9, 1.0):
        m, e, n = orc.group_plan(W, 1, target_fraction=f)
        m2, e2, K = orc.target_fraction(W, f)
        assert (m == m2).all() and e == e2 and n == K


def test_group_plan_shares_one_decision_per_group_and_handles_the_local_state_separately():
    """Section 4.2.1: p/g groups of g adjacent states share one decision; the local state is always
    computed and the group that contains it has g - 1 members.  Measure = sum over the group (Eq. 12)."""
    P, g = 8, 4
    d = np.abs(np.subtract.outer(np.arange(P), np.arange(P))).astype(float)
    W = np.exp(-0.8 * d); W /= W.sum(1, keepdims=True)
    m, eps, n = orc.group_plan(W, g, eps=0.25)
    for i in range(P):
        for k in range(P // g):
            members = [j for j in range(k * g, (k + 1) * g) if j != i]
            assert len(set(m[i, members].tolist())) == 1                         # shared decision
            assert m[i, members[0]] == int(W[i, members].sum() > 0.25)           # Eq. 12 + Eq. 13
            assert len(members) == (g - 1 if i // g == k else g)
    assert (m.diagonal() == 1).all() and n == m.sum()
    # strictness at equality: a measure exactly equal to eps is REUSE
    W2 = np.full((4, 4), 0.25)
    m2, _, _ = orc.group_plan(W2, 2, eps=0.5)      # remote groups sum to exactly 0.5
    assert (m2 == np.eye(4)).all()
    m3, _, _ = orc.group_plan(W2, 2, eps=0.2)      # local groups (one member, 0.25) and remote ones (0.5) exceed it
    assert m3.all()


def test_group_plan_target_fraction_takes_whole_groups_in_rank_order():
    P, g = 8, 2
    d = np.abs(np.subtract.outer(np.arange(P), np.arange(P))).astype(float)
    W = np.exp(-1.1 * d) * (1.0 + 0.02 * np.random.default_rng(16).random((P, P)))   # no tied measures
    W /= W.sum(1, keepdims=True)
    prev = None
    for f in (0.125, 0.3, 0.5, 0.75, 1.0):
        m, eps, n = orc.group_plan(W, g, target_fraction=f)
        K = min(max(int(np.floor(f * P * P + 0.5)), P), P * P)
        assert n == m.sum() and P <= n <= K and (m.diagonal() == 1).all()
        # thresholding the group measures at the reported eps reproduces the selection
        m_thr, _, _ = orc.group_plan(W, g, eps=eps)
        assert (m_thr == m).all()
        if prev is not None:
            assert (m >= prev).all()
        prev = m
    assert orc.group_plan(W, g, target_fraction=1.0)[0].all()


# ---------------------------------------------------------------- Algorithm 1 pieces

def test_scale_ratio_and_state_norm_closed_forms():
    """Eq. 9 on states with known norms: OUT = c_ij everywhere, LSE = 0 -> ||AS(i,j)||^2 = n_i H D c_ij^2,
    so alpha(i,j) = |c_ij| / |c_ii|; scaling every state by the same factor leaves alpha unchanged."""
    P, n, D = 3, 5, 4
    c = np.array([[2.0, 1.0, 0.5], [3.0, 1.5, 6.0], [1.0, 1.0, 1.0]])
    nsq = np.array([[orc.state_norm_sq(np.full((n, D), c[i, j]), np.zeros(n)) for j in range(P)] for i in range(P)])
    np.testing.assert_allclose(nsq, n * D * c * c)
    alpha = orc.scale_ratios(nsq)
    np.testing.assert_allclose(alpha, np.abs(c) / np.abs(np.diag(c))[:, None])
    np.testing.assert_allclose(orc.scale_ratios(9.0 * nsq), alpha)
    assert orc.state_norm_sq(np.zeros((2, 3)), np.array([3.0, 4.0])) == 25.0      # the LSE is part of the state


def test_planner_step_truth_table():
    """Alg. 1: ASE = w * alpha * delta_local summed over the group (Eq. 7, 10, 12); anchor iff every unit
    exceeds eps or the local drift exceeds eps_local (Eq. 14); otherwise COMPUTE iff ASE > eps (Eq. 13)."""
    P = 4
    W = np.array([[0.4, 0.3, 0.2, 0.1], [0.3, 0.4, 0.2, 0.1], [0.1, 0.2, 0.4, 0.3], [0.1, 0.2, 0.3, 0.4]])
    alpha = np.ones((P, P)); alpha[0, 1] = 2.0
    drift = np.array([1.0, 4.0, 0.25, 0.0])          # squared: deltas 1, 2, 0.5, 0
    base = np.full(P, 100.0)
    r = orc.planner_step(W, alpha, drift, base, 1, eps=0.25, eps_local=1.0, R=0.5, have_anchor=True)
    assert not r["is_anchor"]
    np.testing.assert_allclose(r["ase"][0, 1], 0.3 * 2.0 * 1.0)
    np.testing.assert_allclose(r["ase"][1, 0], 0.3 * 2.0)
    np.testing.assert_allclose(r["ase"][2, 3], 0.3 * 0.5)
    assert np.isnan(r["ase"][2, 2]) and (r["ase"][3, :3] == 0).all()
    expect = np.eye(P, dtype=np.uint8)
    expect[0, 1] = 1                                   # 0.6 > 0.25 ; (0,2) = 0.2, (0,3) = 0.1 reuse
    expect[1, 0] = expect[1, 2] = 1                    # 0.6, 0.4 ; (1,3) = 0.2 reuse
    assert (r["mask"] == expect).all() and r["eps"] == 0.25
    assert r["delta_rel"] == pytest.approx(np.sqrt(5.25 / 400.0))
    # the local drift alone triggers an anchor
    r2 = orc.planner_step(W, alpha, drift, base, 1, eps=0.25, eps_local=0.1, R=0.5, have_anchor=True)
    assert r2["is_anchor"] and r2["mask"].all()
    # eps becomes the R-quantile of the predicted unit errors: half of the 12 units at or below it
    vals = np.sort(r["ase"][~np.isnan(r["ase"])])
    assert r2["eps"] == pytest.approx(0.5 * (vals[5] + vals[6]))
    assert (vals <= r2["eps"]).sum() == 6
    # every unit above eps -> anchor; strictness: a unit exactly at eps is not "above"
    r3 = orc.planner_step(W, alpha, np.full(P, 1.0), base, 1, eps=0.05, eps_local=10.0, R=0.5, have_anchor=True)
    assert r3["is_anchor"]
    r4 = orc.planner_step(W, alpha, np.full(P, 1.0), base, 1, eps=0.1, eps_local=10.0, R=0.5, have_anchor=True)
    assert not r4["is_anchor"] and r4["mask"][0, 3] == 0 and r4["mask"][0, 2] == 1
    # no anchor yet -> the first step is one, and eps is kept when nothing has drifted
    r5 = orc.planner_step(W, alpha, np.zeros(P), base, 1, eps=0.3, eps_local=1.0, R=0.5, have_anchor=False)
    assert r5["is_anchor"] and r5["eps"] == 0.3
    # groups: the unit's error is the sum over its members, the local member excluded
    r6 = orc.planner_step(W, alpha, drift, base, 2, eps=0.25, eps_local=1.0, R=0.5, have_anchor=True)
    np.testing.assert_allclose(r6["ase"][0, 0], 0.6)              # only j = 1 (j = 0 is local)
    np.testing.assert_allclose(r6["ase"][0, 1], 0.2 + 0.1)
    np.testing.assert_allclose(r6["ase"][1, 1], (0.2 + 0.1) * 2.0)
    assert r6["mask"][1].tolist() == [1, 1, 1, 1] and r6["mask"][0].tolist() == [1, 1, 1, 1] and r6["mask"][2].tolist() == [0, 0, 1, 0]


def test_uniform_offsets():
    off = orc.uniform_offsets(32760, 16)
    assert off[0] == 0 and off[-1] == 32760
    sizes = np.diff(off)
    assert set(sizes.tolist()) == {2047, 2048} and (sizes == 2047).sum() == 8


# ---------------------------------------------------------------- input widening (bf16 / fp16)

def test_widening_of_every_16_bit_pattern_is_exact():
    """The oracle computes with the exact value of each input element: all 65 536 bit patterns of both input
    types against numpy / torch conversions (subnormals, infinities and NaN included)."""
    bits = np.arange(65536, dtype=np.uint16)
    ref16 = bits.view(np.float16).astype(np.float64)
    refbf = widen(bits)
    for b in range(0, 65536, 1):
        g16, gbf = orc.widen(b, fp16=True), orc.widen(b, fp16=False)
        assert (math.isnan(g16) and math.isnan(ref16[b])) or g16 == ref16[b], hex(b)
        assert (math.isnan(gbf) and math.isnan(refbf[b])) or gbf == refbf[b], hex(b)
        if b % 97:          # the full sweep of the cheap comparison above, the sign check on a subset
            continue
        assert math.isnan(g16) or math.copysign(1.0, g16) == math.copysign(1.0, float(ref16[b]))


def test_fp16_inputs_full_attention_matches_library_sdpa():
    """Table 1 (the Wan models run in FP16): the same definitions on fp16 bit patterns."""
    rng = np.random.default_rng(12)
    B, L, H, D = 1, 29, 2, 16
    x = [rng.standard_normal((B, L, H, D)).astype(np.float16) for _ in range(3)]
    q, k, v = (a.view(np.uint16).copy() for a in x)
    qt, kt, vt = (torch.from_numpy(a.astype(np.float64)).permute(0, 2, 1, 3) for a in x)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=0.3).numpy()
    off = orc.uniform_offsets(L, 3)
    for h in range(H):
        o, lse = orc.full_attention(q, k, v, 0.3, 0, h, all_rows(L), fp16=True)
        np.testing.assert_allclose(o, ref[0, h], rtol=0, atol=1e-13)
        ses = orc.OracleSession(B, L, H, D, off, 0.3, {(0, h): all_rows(L)}, fp16=True)
        outs, _ = ses.step(q, k, v, np.ones((3, 3), np.uint8), 0)
        np.testing.assert_allclose(outs[(0, h)], ref[0, h], rtol=0, atol=1e-13)
    # the same bits read as bf16 give a different answer: the flag is not ignored
    o_bf, _ = orc.full_attention(q, k, v, 0.3, 0, 0, all_rows(L), fp16=False)
    assert np.abs(o_bf - ref[0, 0]).max() > 1e-3


def test_config0_regression_values():
    """The oracle and the seeded inputs reproduce the committed summary values of the correctness configuration
    (regression only: written by tests/golden/make_config0_reference.py from the oracle itself)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_config0_reference", os.path.join(GOLDEN, "make_config0_reference.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = [l.strip() for l in open(os.path.join(GOLDEN, "config0_reference.txt")) if not l.startswith("#")]
    got = mod.summarise()
    assert len(got) == len(want)
    for g, w in zip(got, want):
        gt, wt = g.split(), w.split()
        assert len(gt) == len(wt)
        for a, b in zip(gt, wt):
            try:
                fa, fb = float(a), float(b)
            except ValueError:
                assert a == b
                continue
            assert fa == pytest.approx(fb, rel=1e-9, abs=1e-12), (g, w)
