"""Seeded workload generator: determinism, shapes, and the distance-decaying partition
contribution that the paper reports for video DiTs (Fig. 2 / Fig. 5)."""
import numpy as np
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import inputs


def test_workload_shapes_match_named_configs():
    w = inputs.WORKLOADS
    assert w["c0_correctness"].L == 1024 and w["c1_cogvideox"].L == 17776
    assert w["c2_wan480p"].L == 32760 and w["c3_wan720p"].L == 75600 and w["c4_hunyuan720p"].L == 118800
    assert np.diff(w["c1_cogvideox"].offsets()).tolist() == [2222] * 8
    assert set(np.diff(w["c4_hunyuan720p"].offsets()).tolist()) == {3712, 3713}
    assert inputs.banded_mask(4).sum() == 10


def test_generator_is_deterministic_and_steps_differ():
    wl = inputs.tiny_workload(grid=(2, 5, 6), n_text=3, H=2, D=64)
    a, b = inputs.StepInputs(wl, seed=3), inputs.StepInputs(wl, seed=3)
    q1, k1, v1 = a.next()
    q1b, _, _ = b.next()
    assert q1.dtype == torch.bfloat16 and tuple(q1.shape) == (1, wl.L, 2, 64)
    assert torch.equal(q1, q1b)
    q2, _, _ = a.next()
    d = (q2.float() - q1.float()).abs().mean().item()
    assert 0.01 < d < 0.1                      # sigma 0.05 perturbation, bf16-rounded
    qc, _, _ = inputs.StepInputs(wl, seed=4).next()
    assert not torch.equal(q1, qc)
    assert inputs.bf16_bits(q1).dtype == np.uint16


def test_partition_contribution_decays_with_distance():
    """Mean contribution W by |i - j| falls with distance (the locality the workloads imitate)."""
    wl = inputs.Workload("probe", 1, 1, 64, (8, 12, 12), 0, 8, 1, 0.05)
    q, k, v = (inputs.bf16_bits(t) for t in inputs.StepInputs(wl, seed=0).next())
    off = wl.offsets()
    rows = np.arange(0, wl.L, 3, dtype=np.int32)
    lse = np.full((wl.P, 1, 1, wl.L), 0.0)
    for j in range(wl.P):
        lse[j, 0, 0, rows] = orc.pair_state(q, k, v, wl.scale, 0, 0, rows, off[j], off[j + 1])[1]
    # rows not sampled get a constant LSE on every partition (uniform weights) -- exclude them
    sub = lse[:, :, :, rows]
    part = np.searchsorted(off, rows, side="right") - 1
    sm = np.exp(sub - np.log(np.exp(sub).sum(0, keepdims=True)))[:, 0, 0, :]      # [P, nrows]
    by_dist = [np.mean([sm[j, r] for r in range(rows.size) for j in range(wl.P) if abs(part[r] - j) == d])
               for d in range(4)]
    assert by_dist[0] > by_dist[1] > by_dist[2] > by_dist[3]


def test_sample_rows_cover_boundaries():
    wl = inputs.WORKLOADS["c0_correctness"]
    rows = inputs.sample_rows(wl, 64, seed=1)
    allr = set(int(r) for v in rows.values() for r in v)
    assert {0, wl.L - 1, 256, 255, 512, 767} <= allr
    assert all(0 <= b < wl.B and 0 <= h < wl.H for b, h in rows)
