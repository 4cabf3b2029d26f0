"""Python face of the fp64 CPU oracle (ctypes marshalling + the per-step cache semantics).

TEST INFRASTRUCTURE ONLY -- see oracle/__init__.py.  All arithmetic of Eq. 1, Eq. 2,
Eq. 8 and Eq. 13 lives in ditango_oracle.c; this file only moves numpy arrays in and out
and keeps the state cache of the selective compute / reuse step (Section 2.2.4, Fig. 6;
cache timestep t_c of Section 4.2.2; Algorithm 1's t_c bookkeeping).

Q, K, V are numpy uint16 arrays holding bf16 (or, with fp16=True, IEEE fp16) bit patterns in layout [B, L, H, D].
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        u16p, i32p, f64p, u8p = (C.POINTER(C.c_uint16), C.POINTER(C.c_int32),
                                 C.POINTER(C.c_double), C.POINTER(C.c_uint8))
        L.orc_num_threads.restype = C.c_int
        L.orc_pair_state.restype = C.c_int
        L.orc_pair_state.argtypes = [u16p, u16p, u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double,
                                     C.c_int, C.c_int, i32p, C.c_int, C.c_int, C.c_int, f64p, f64p, C.c_int]
        L.orc_widen.restype = C.c_double
        L.orc_widen.argtypes = [C.c_uint16, C.c_int]
        L.orc_full_attention.restype = C.c_int
        L.orc_full_attention.argtypes = [u16p, u16p, u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double,
                                         C.c_int, C.c_int, i32p, C.c_int, f64p, f64p, C.c_int]
        L.orc_compose2.restype = None
        L.orc_compose2.argtypes = [f64p, C.c_double, f64p, C.c_double, C.c_int, f64p, f64p]
        L.orc_merge.restype = None
        L.orc_merge.argtypes = [f64p, f64p, C.c_int, C.c_int, C.c_int, f64p, f64p]
        L.orc_contribution.restype = C.c_int
        L.orc_contribution.argtypes = [f64p, C.c_int, C.c_int, C.c_int, C.c_int, i32p, f64p]
        L.orc_threshold.restype = None
        L.orc_threshold.argtypes = [f64p, C.c_int, C.c_double, u8p]
        L.orc_target_fraction.restype = C.c_int
        L.orc_target_fraction.argtypes = [f64p, C.c_int, C.c_double, u8p, f64p]
        L.orc_group_plan.restype = C.c_int
        L.orc_group_plan.argtypes = [f64p, C.c_int, C.c_int, C.c_double, C.c_double, u8p, f64p]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _chk_qkv(q, k, v):
    for t in (q, k, v):
        if t.dtype != np.uint16 or t.ndim != 4 or not t.flags.c_contiguous:
            raise ValueError("q, k, v must be C-contiguous uint16 (bf16 bits) arrays [B, L, H, D]")
    if not (q.shape == k.shape == v.shape):
        raise ValueError("q, k, v shapes differ")
    return q.shape


def widen(bits, fp16=False):
    """One 16-bit pattern (bf16, or IEEE fp16) as the double the oracle computes with."""
    return float(lib().orc_widen(int(bits), 1 if fp16 else 0))


def pair_state(q, k, v, scale, b, h, rows, key_begin, key_end, fp16=False):
    """Eq. 1 for the listed query rows of (b, h) against keys [key_begin, key_end).
    q, k, v hold bf16 bit patterns, or fp16 ones with fp16=True (Table 1: the Wan models run in FP16).

    Returns (OUT [nrows, D], LSE [nrows]) in fp64."""
    B, L, H, D = _chk_qkv(q, k, v)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    out = np.empty((rows.size, D), dtype=np.float64)
    lse = np.empty((rows.size,), dtype=np.float64)
    rc = lib().orc_pair_state(_p(q, C.c_uint16), _p(k, C.c_uint16), _p(v, C.c_uint16), B, L, H, D,
                              float(scale), int(b), int(h), _p(rows, C.c_int32), rows.size,
                              int(key_begin), int(key_end), _p(out, C.c_double), _p(lse, C.c_double), 1 if fp16 else 0)
    if rc != 0:
        raise ValueError("orc_pair_state: bad arguments")
    return out, lse


def full_attention(q, k, v, scale, b, h, rows, fp16=False):
    """softmax(scale * q K^T) V over all L keys for the listed rows of (b, h), fp64."""
    B, L, H, D = _chk_qkv(q, k, v)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    out = np.empty((rows.size, D), dtype=np.float64)
    lse = np.empty((rows.size,), dtype=np.float64)
    rc = lib().orc_full_attention(_p(q, C.c_uint16), _p(k, C.c_uint16), _p(v, C.c_uint16), B, L, H, D,
                                  float(scale), int(b), int(h), _p(rows, C.c_int32), rows.size,
                                  _p(out, C.c_double), _p(lse, C.c_double), 1 if fp16 else 0)
    if rc != 0:
        raise ValueError("orc_full_attention: bad arguments")
    return out, lse


def compose2(oa, lsea, ob, lseb):
    """Eq. 2 for two states of one query row."""
    oa = np.ascontiguousarray(oa, dtype=np.float64)
    ob = np.ascontiguousarray(ob, dtype=np.float64)
    o = np.empty_like(oa)
    lse = C.c_double()
    lib().orc_compose2(_p(oa, C.c_double), float(lsea), _p(ob, C.c_double), float(lseb), oa.size,
                       _p(o, C.c_double), C.byref(lse))
    return o, lse.value


def merge(o_states, lse_states):
    """Eq. 2 folded over P states per row: o_states [n, P, D], lse_states [n, P]."""
    o_states = np.ascontiguousarray(o_states, dtype=np.float64)
    lse_states = np.ascontiguousarray(lse_states, dtype=np.float64)
    n, P, D = o_states.shape
    assert lse_states.shape == (n, P)
    out = np.empty((n, D), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    lib().orc_merge(_p(o_states, C.c_double), _p(lse_states, C.c_double), n, P, D,
                    _p(out, C.c_double), _p(lse, C.c_double))
    return out, lse


def contribution(lse_states, off):
    """Eq. 8 per row, averaged to W[i][j]; lse_states [P, B, H, L] fp64, off [P+1]."""
    lse_states = np.ascontiguousarray(lse_states, dtype=np.float64)
    P, B, H, L = lse_states.shape
    off = np.ascontiguousarray(off, dtype=np.int32)
    assert off.size == P + 1
    W = np.empty((P, P), dtype=np.float64)
    rc = lib().orc_contribution(_p(lse_states, C.c_double), B, H, L, P, _p(off, C.c_int32), _p(W, C.c_double))
    if rc != 0:
        raise ValueError("orc_contribution: bad partition offsets")
    return W


def threshold(W, eps):
    """Eq. 13 with the diagonal forced to COMPUTE; returns uint8 [P, P]."""
    W = np.ascontiguousarray(W, dtype=np.float64)
    P = W.shape[0]
    mask = np.empty((P, P), dtype=np.uint8)
    lib().orc_threshold(_p(W, C.c_double), P, float(eps), _p(mask, C.c_uint8))
    return mask


def target_fraction(W, f):
    """Percentile choice of eps for a target computed-pair fraction; returns (mask, eps, K)."""
    W = np.ascontiguousarray(W, dtype=np.float64)
    P = W.shape[0]
    mask = np.empty((P, P), dtype=np.uint8)
    eps = C.c_double()
    K = lib().orc_target_fraction(_p(W, C.c_double), P, float(f), _p(mask, C.c_uint8), C.byref(eps))
    return mask, eps.value, int(K)


def group_plan(W, g, eps=0.0, target_fraction=-1.0):
    """Group-wise decisions (Section 4.2.1-4.2.3): one decision per (query partition, group of g KV
    partitions), diagonal always computed.  Returns (mask, eps_used, computed_pairs)."""
    W = np.ascontiguousarray(W, dtype=np.float64)
    P = W.shape[0]
    mask = np.empty((P, P), dtype=np.uint8)
    eps_out = C.c_double()
    n = lib().orc_group_plan(_p(W, C.c_double), P, int(g), float(eps), float(target_fraction), _p(mask, C.c_uint8),
                             C.byref(eps_out))
    return mask, eps_out.value, int(n)


def uniform_offsets(L, P):
    """off_p = floor(p L / P): contiguous partitions whose sizes differ by at most one."""
    return np.array([(p * L) // P for p in range(P + 1)], dtype=np.int32)


class OracleSession:
    """Selective compute / reuse over denoising steps for a chosen set of query rows.

    The cache holds, per (query row, KV partition j), the state of the last step at which
    the pair (partition of the row, j) was computed (t_c); it starts empty (t_c = -1).
    step(): COMPUTE pairs are recomputed from the step's inputs (Eq. 1) and overwrite
    their slots; REUSE pairs keep their slots (an empty one is an error); the output is
    the composition of all P slots (Eq. 2).

    rows_by_bh: dict {(b, h): int array of query rows}; only these rows are evaluated,
    which is what lets large workloads be checked on a sample.
    """

    def __init__(self, B, L, H, D, off, scale, rows_by_bh, fp16=False):
        self.B, self.L, self.H, self.D = B, L, H, D
        self.fp16 = bool(fp16)
        self.off = np.ascontiguousarray(off, dtype=np.int32)
        self.P = self.off.size - 1
        self.scale = float(scale)
        self.rows = {bh: np.ascontiguousarray(r, dtype=np.int32) for bh, r in rows_by_bh.items()}
        self.part = {bh: np.searchsorted(self.off, r, side="right") - 1 for bh, r in self.rows.items()}
        self.o = {bh: np.zeros((r.size, self.P, D)) for bh, r in self.rows.items()}
        self.lse = {bh: np.zeros((r.size, self.P)) for bh, r in self.rows.items()}
        self.tc = -np.ones((self.P, self.P), dtype=np.int32)

    def step(self, q, k, v, mask, t):
        mask = np.asarray(mask).reshape(self.P, self.P)
        for i in range(self.P):
            for j in range(self.P):
                if not mask[i, j] and self.tc[i, j] < 0:
                    raise RuntimeError(f"REUSE of pair ({i},{j}) that was never computed")
        outs, lses = {}, {}
        for bh, rows in self.rows.items():
            b, h = bh
            for i in range(self.P):
                sel = np.nonzero(self.part[bh] == i)[0]
                if sel.size == 0:
                    continue
                for j in range(self.P):
                    if mask[i, j]:
                        o, l = pair_state(q, k, v, self.scale, b, h, rows[sel],
                                          int(self.off[j]), int(self.off[j + 1]), fp16=self.fp16)
                        self.o[bh][sel, j, :] = o
                        self.lse[bh][sel, j] = l
            outs[bh], lses[bh] = merge(self.o[bh], self.lse[bh])
        self.tc[mask.astype(bool)] = t
        return outs, lses


# --------------------------------------------------------------------------------------------------
# Anchor-guided selection planning (Section 4; Algorithm 1), in plain numpy fp64.
#
# Readings where the paper is silent:
#   * ||AS||_2 (Eq. 9, Eq. 10) is the 2-norm of OUT and LSE stacked, taken over all rows and heads of the
#     query partition;
#   * delta(j, t, t_c) is evaluated against the last anchor for every state (Eq. 10 defines it only for
#     t_a), t_c is bookkeeping;
#   * delta_local(t) of Eq. 14 is the relative change of the local states over all query partitions:
#     sqrt(sum_i ||AS_t(i,i) - AS_ta(i,i)||^2) / sqrt(sum_i ||AS_ta(i,i)||^2);
#   * "update eps based on R and anchor errors": eps becomes the R-quantile of the units' predicted ASE at
#     the step that turned into an anchor (fraction R of the units would have been reused under that
#     drift); it is left unchanged when those values are all zero (the very first anchor);
#   * the first step is an anchor.
# These parts are pinned only by closed forms and invariants ("parity unpinned" for the readings).

def state_norm_sq(o, lse):
    """||AS||_2^2 of a set of rows: OUT [n, D] and LSE [n] stacked (Eq. 1's AS)."""
    o = np.asarray(o, dtype=np.float64); lse = np.asarray(lse, dtype=np.float64)
    return float((o * o).sum() + (lse * lse).sum())


def scale_ratios(norm_sq):
    """Eq. 9: alpha(i, j) = ||AS_ta(i, j)||_2 / ||AS_ta(i, i_loc)||_2 with the local state on the diagonal."""
    n = np.asarray(norm_sq, dtype=np.float64)
    return np.sqrt(n / np.diag(n)[:, None])


def planner_step(W, alpha, drift_sq, anchor_local_sq, g, eps, eps_local, R, have_anchor):
    """One pass of Algorithm 1 given this step's local states.
    drift_sq[i] = ||AS_t(i,i) - AS_ta(i,i)||^2, anchor_local_sq[i] = ||AS_ta(i,i)||^2.
    Returns dict(is_anchor, mask [P,P] uint8 with the diagonal set, ase [P, n_groups] (nan where a unit
    has no member), eps (possibly updated), delta_rel)."""
    W = np.asarray(W, dtype=np.float64); alpha = np.asarray(alpha, dtype=np.float64)
    P = W.shape[0]
    g = max(1, int(g))
    ng = (P + g - 1) // g
    delta = np.sqrt(np.asarray(drift_sq, dtype=np.float64))
    ase = np.full((P, ng), np.nan)
    for i in range(P):
        for k in range(ng):
            members = [j for j in range(k * g, min(P, (k + 1) * g)) if j != i]
            if members:
                s = 0.0
                for j in members:                                  # Eq. 7, Eq. 10, Eq. 12
                    s += W[i, j] * alpha[i, j] * delta[i]
                ase[i, k] = s
    valid = ~np.isnan(ase)
    vals = ase[valid]
    den = float(np.sum(anchor_local_sq))
    delta_rel = float(np.sqrt(np.sum(drift_sq) / den)) if den > 0 else 0.0
    all_exceed = bool(vals.size > 0 and (vals > eps).all())
    local_drift = delta_rel > eps_local
    is_anchor = (not have_anchor) or all_exceed or local_drift      # Eq. 14; the first step is an anchor
    mask = np.eye(P, dtype=np.uint8)
    eps_new = eps
    if is_anchor:
        mask[:] = 1
        if vals.size > 0 and vals.max() > 0.0:
            a = np.sort(vals)
            r = int(np.floor(R * a.size))
            r = min(max(r, 0), a.size)
            eps_new = 0.0 if r == 0 else (float(a[-1]) if r == a.size else 0.5 * float(a[r - 1] + a[r]))
    else:
        for i in range(P):
            for j in range(P):
                if i != j and ase[i, j // g] > eps:                # Eq. 13, strict
                    mask[i, j] = 1
    return dict(is_anchor=bool(is_anchor), mask=mask, ase=ase, eps=float(eps_new), delta_rel=delta_rel)


# --------------------------------------------------------------------------------------------------
# Grouped state cache (Section 4.2.1, Section 4.2.2; Dynamic Group State Compose, Eq. 15).
#
# The P states of a query partition i are organised as m = ceil(P / g) groups of g adjacent KV partitions
# plus the local state, which is handled separately: slot 0 = local state (i, i); slot 1 + k = AS(G_k), the
# composition (Eq. 2) of the states of group k's partitions, without partition i in the group that holds it.
# Everything here is written as that definition: a group state is computed member by member (Eq. 1) and
# composed with `merge` (Eq. 2); nothing evaluates a group in one pass.

def group_slots(P, g):
    """members[i][s]: KV partitions behind slot s of query partition i (an empty list: no such slot)."""
    g = max(1, int(g))
    m = (P + g - 1) // g
    return [[[i]] + [[j for j in range(k * g, min(P, (k + 1) * g)) if j != i] for k in range(m)] for i in range(P)]


def slot_contribution(lse_slots, off, members):
    """Importance of every slot (Eq. 8 summed over the slot's members, Eq. 12): per query row the softmax of
    the slots' LSEs, averaged over batch, heads and the rows of query partition i.  lse_slots [S, B, H, L]."""
    lse_slots = np.asarray(lse_slots, dtype=np.float64)
    S = lse_slots.shape[0]
    P = len(off) - 1
    W = np.zeros((P, S))
    for i in range(P):
        x = lse_slots[:, :, :, off[i]:off[i + 1]].copy()
        for s in range(S):
            if not members[i][s]:
                x[s] = -np.inf
        mx = x.max(axis=0, keepdims=True)
        e = np.exp(x - mx)
        w = e / e.sum(axis=0, keepdims=True)
        W[i] = w.reshape(S, -1).mean(axis=1)
    return W


def slot_plan(W, members, g, eps=0.0, target_fraction=-1.0):
    """One decision per non-local slot that exists (Section 4.2.3): COMPUTE iff W > eps (Eq. 13, strict), or,
    for target_fraction >= 0, slots in order of decreasing W (ties: the group nearer to the local one, then
    the smaller flat index i * S + s) while their members fit into K - P pairs, K = round(f P^2) clipped to
    [P, P^2].  The local slot 0 is always COMPUTE.  Returns (mask [P, S] uint8, eps_used)."""
    W = np.asarray(W, dtype=np.float64)
    P, S = W.shape
    mask = np.zeros((P, S), dtype=np.uint8)
    mask[:, 0] = 1
    units = [(i, s) for i in range(P) for s in range(1, S) if members[i][s]]
    if target_fraction < 0:
        for i, s in units:
            if W[i, s] > eps:
                mask[i, s] = 1
        return mask, float(eps)
    K = int(np.floor(target_fraction * P * P + 0.5))
    K = min(max(K, P), P * P)
    budget = K - P
    order = sorted(units, key=lambda u: (-W[u], abs((u[1] - 1) - u[0] // g), u[0] * S + u[1]))
    cum, taken = 0, 0
    for r, u in enumerate(order):        # a unit is taken iff it and everything ranked before it fit
        cum += len(members[u[0]][u[1]])
        if cum <= budget:
            mask[u] = 1
            taken = r + 1
    if not order or taken == len(order):
        eps_used = 0.0
    elif taken == 0:
        eps_used = float(W[order[0]])
    else:
        eps_used = 0.5 * float(W[order[taken - 1]] + W[order[taken]])
    return mask, eps_used


class GroupedOracleSession:
    """OracleSession for a grouped cache: per (query row, slot) the cached group state; COMPUTE slots are
    recomputed member by member (Eq. 1) and composed (Eq. 2); the output composes all slots that exist.
    compose() is Dynamic Group State Compose with k = 2 (Eq. 15); reset() returns to the original g."""

    def __init__(self, B, L, H, D, off, scale, rows_by_bh, g, fp16=False):
        self.B, self.L, self.H, self.D = B, L, H, D
        self.fp16 = bool(fp16)
        self.off = np.ascontiguousarray(off, dtype=np.int32)
        self.P = self.off.size - 1
        self.scale = float(scale)
        self.g0 = int(g)
        self.rows = {bh: np.ascontiguousarray(r, dtype=np.int32) for bh, r in rows_by_bh.items()}
        self.part = {bh: np.searchsorted(self.off, r, side="right") - 1 for bh, r in self.rows.items()}
        self._layout(self.g0)
        self.o = {bh: np.zeros((r.size, self.S, D)) for bh, r in self.rows.items()}
        self.lse = {bh: np.full((r.size, self.S), -np.inf) for bh, r in self.rows.items()}
        self.tc = -np.ones((self.P, self.S), dtype=np.int32)

    def _layout(self, g):
        self.g = g
        self.members = group_slots(self.P, g)
        self.S = len(self.members[0])

    def step(self, q, k, v, mask, t):
        mask = np.asarray(mask).reshape(self.P, self.S)
        for i in range(self.P):
            for s in range(self.S):
                if self.members[i][s] and not mask[i, s] and self.tc[i, s] < 0:
                    raise RuntimeError(f"REUSE of slot ({i},{s}) that was never computed")
        outs, lses = {}, {}
        for bh, rows in self.rows.items():
            b, h = bh
            for i in range(self.P):
                sel = np.nonzero(self.part[bh] == i)[0]
                if sel.size == 0:
                    continue
                for s in range(self.S):
                    mem = self.members[i][s]
                    if not mem or not mask[i, s]:
                        continue
                    po = np.empty((sel.size, len(mem), self.D)); pl = np.empty((sel.size, len(mem)))
                    for a, j in enumerate(mem):                    # Eq. 1 per member partition
                        po[:, a, :], pl[:, a] = pair_state(q, k, v, self.scale, b, h, rows[sel],
                                                           int(self.off[j]), int(self.off[j + 1]), fp16=self.fp16)
                    self.o[bh][sel, s, :], self.lse[bh][sel, s] = merge(po, pl)   # Eq. 2: the group state
            outs[bh], lses[bh] = merge(self.o[bh], self.lse[bh])
        for i in range(self.P):
            for s in range(self.S):
                if self.members[i][s] and mask[i, s]:
                    self.tc[i, s] = t
        return outs, lses

    def compose(self):
        """Eq. 15, k = 2: AS(G_2k) (+) AS(G_2k+1) -> AS(G'_k); the local slot stays."""
        S_old, old_members = self.S, self.members
        self._layout(self.g * 2)
        for bh in self.rows:
            o_old, l_old = self.o[bh], self.lse[bh]
            o_new = np.zeros((o_old.shape[0], self.S, self.D)); l_new = np.full((o_old.shape[0], self.S), -np.inf)
            o_new[:, 0], l_new[:, 0] = o_old[:, 0], l_old[:, 0]
            for s in range(1, self.S):
                src = [x for x in (2 * s - 1, 2 * s) if x < S_old]
                o_new[:, s], l_new[:, s] = merge(o_old[:, src, :], l_old[:, src])
            self.o[bh], self.lse[bh] = o_new, l_new
        tc_new = -np.ones((self.P, self.S), dtype=np.int32)
        tc_new[:, 0] = self.tc[:, 0]
        for i in range(self.P):
            for s in range(1, self.S):
                src = [x for x in (2 * s - 1, 2 * s) if x < S_old and old_members[i][x]]
                tc_new[i, s] = min(self.tc[i, x] for x in src) if src else -1
        self.tc = tc_new

    def reset(self):
        self._layout(self.g0)
        for bh, r in self.rows.items():
            self.o[bh] = np.zeros((r.size, self.S, self.D))
            self.lse[bh] = np.full((r.size, self.S), -np.inf)
        self.tc = -np.ones((self.P, self.S), dtype=np.int32)


def planner_step_slots(W, alpha, members, drift_sq, anchor_local_sq, eps, eps_local, R, have_anchor):
    """Algorithm 1 on a grouped cache: one unit per non-local slot that exists; a group state is one state, so
    ASE(i, s) = W[i, s] * alpha[i, s] * delta(i) (Eq. 7, Eq. 10, Eq. 12 with the group as its single member).
    Same anchor test (Eq. 14), threshold (Eq. 13) and eps update as planner_step.
    Returns dict(is_anchor, mask [P, S], ase [P, S] (nan where there is no unit), eps, delta_rel)."""
    W = np.asarray(W, dtype=np.float64); alpha = np.asarray(alpha, dtype=np.float64)
    P, S = W.shape
    delta = np.sqrt(np.asarray(drift_sq, dtype=np.float64))
    ase = np.full((P, S), np.nan)
    for i in range(P):
        for s in range(1, S):
            if members[i][s]:
                ase[i, s] = W[i, s] * alpha[i, s] * delta[i]
    vals = ase[~np.isnan(ase)]
    den = float(np.sum(anchor_local_sq))
    delta_rel = float(np.sqrt(np.sum(drift_sq) / den)) if den > 0 else 0.0
    all_exceed = bool(vals.size > 0 and (vals > eps).all())
    is_anchor = (not have_anchor) or all_exceed or (delta_rel > eps_local)
    mask = np.zeros((P, S), dtype=np.uint8)
    mask[:, 0] = 1
    eps_new = eps
    if is_anchor:
        mask[:] = 1
        if vals.size > 0 and vals.max() > 0.0:
            a = np.sort(vals)
            r = min(max(int(np.floor(R * a.size)), 0), a.size)
            eps_new = 0.0 if r == 0 else (float(a[-1]) if r == a.size else 0.5 * float(a[r - 1] + a[r]))
    else:
        for i in range(P):
            for s in range(1, S):
                if members[i][s] and ase[i, s] > eps:
                    mask[i, s] = 1
    return dict(is_anchor=bool(is_anchor), mask=mask, ase=ase, eps=float(eps_new), delta_rel=delta_rel)
