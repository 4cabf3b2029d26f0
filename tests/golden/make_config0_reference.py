"""Writes tests/golden/config0_reference.txt: summary values of the ORACLE's outputs on the correctness
configuration (c0_correctness: 1024 tokens, 2 heads, D 64, P 4; step 1 all pairs, step 2 the band |i-j| <= 1).

These are regression values of the oracle itself (the paper prints no numeric example): they catch an
accidental change of the oracle or of the input generator, they are not independent truth.  Only `oracle/` and
the seeded input generator are used -- nothing from the CUDA path.

    python tests/golden/make_config0_reference.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import oracle as orc  # noqa: E402
from paper_2607_15650_b200 import inputs  # noqa: E402


def summarise():
    wl = inputs.WORKLOADS["c0_correctness"]
    off = wl.offsets()
    rows = {(0, h): np.arange(wl.L, dtype=np.int32) for h in range(wl.H)}
    ses = orc.OracleSession(wl.B, wl.L, wl.H, wl.D, off, wl.scale, rows)
    gen = inputs.StepInputs(wl, seed=0, device="cpu")
    lines = []
    for t, mask in ((1, np.ones((wl.P, wl.P), np.uint8)), (2, inputs.banded_mask(wl.P, 1))):
        q, k, v = gen.next()
        outs, lses = ses.step(*(inputs.bf16_bits(x) for x in (q, k, v)), mask, t)
        for h in range(wl.H):
            o, l = outs[(0, h)], lses[(0, h)]
            lines.append(f"step {t} head {h} out_sum {o.sum():.12e} out_abs_sum {np.abs(o).sum():.12e} "
                         f"out_row500_col7 {o[500, 7]:.12e} lse_sum {l.sum():.12e} lse_row1023 {l[1023]:.12e}")
        lse_all = np.stack([np.stack([ses.lse[(0, h)][:, j] for h in range(wl.H)]) for j in range(wl.P)])[:, None]
        W = orc.contribution(lse_all, off)
        lines.append(f"step {t} W " + " ".join(f"{x:.12e}" for x in W.reshape(-1)))
    return lines


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config0_reference.txt")
    with open(path, "w") as fh:
        fh.write("# oracle regression values for c0_correctness; written by make_config0_reference.py\n")
        fh.write("\n".join(summarise()) + "\n")
    print("wrote", path)
