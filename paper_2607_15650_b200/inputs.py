"""Seeded synthetic workloads shaped like video-DiT attention inputs.

This module serves both the CUDA path's tests / benchmark and the CPU oracle's tests.  It
holds none of the method's arithmetic: only shapes, partition offsets, random tensors and
row sampling.

Recipe (all draws from torch generators seeded from `seed` and a fixed stream id):
  * tokens are a (t, h, w) grid flattened row-major, optionally preceded by text tokens;
  * feature map phi(x) in R^16, phi_m = cos(omega_m . x + theta_m), omega_m ~ U(0, 0.3)^3
    rad/token, theta_m ~ U(0, 2 pi), shared by all heads and by Q, K, V;
  * per head a projection A_h in R^{16 x D}, entries N(0, variance 1/16); Q and K share
    A_h (that is what gives nearby tokens large logits), V has its own;
  * video rows: X = 0.6 N(0,1) + phi(x)^T A_h;  text rows: N(0,1);  fp32 masters;
  * step s+1 masters = step s masters + sigma N(0,1); each step's masters are rounded to
    bf16 (round-to-nearest-even);  softmax scale 1/sqrt(D).
These stand in for the Q/K/V activations of the video DiTs the paper evaluates
(Table 1): same tensor shapes and the distance-decaying partition contribution of
Fig. 2 / Fig. 5, not the models' values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

N_FEATURES = 16
STREAM_FEATURES, STREAM_PROJ_QK, STREAM_PROJ_V, STREAM_NOISE, STREAM_STEP, STREAM_ROWS = 1, 2, 3, 4, 5, 6


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    D: int
    grid: tuple            # (T, Hg, Wg) video token grid
    n_text: int
    P: int
    steps: int
    sigma: float
    fractions: tuple = field(default=(1.0,))   # computed-pair fractions the workload sweeps

    @property
    def L(self) -> int:
        return self.n_text + self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    def offsets(self) -> np.ndarray:
        """off_p = floor(p L / P): contiguous partitions, sizes differ by at most one."""
        return np.array([(p * self.L) // self.P for p in range(self.P + 1)], dtype=np.int32)


WORKLOADS = {
    "c0_correctness": Workload("c0_correctness", 1, 2, 64, (4, 16, 16), 0, 4, 2, 0.05, (1.0, 0.625)),
    "c1_cogvideox": Workload("c1_cogvideox", 1, 48, 64, (13, 30, 45), 226, 8, 4, 0.05, (1.0, 0.5)),
    "c2_wan480p": Workload("c2_wan480p", 1, 40, 128, (21, 30, 52), 0, 16, 4, 0.05, (1.0, 0.5, 0.25)),
    "c3_wan720p": Workload("c3_wan720p", 1, 40, 128, (21, 45, 80), 0, 16, 8, 0.03, (1.0, 0.4)),
    "c4_hunyuan720p": Workload("c4_hunyuan720p", 1, 24, 128, (33, 45, 80), 0, 32, 4, 0.05,
                               (1.0, 0.5, 0.25, 0.125)),
}


def tiny_workload(name="tiny", B=1, H=2, D=64, grid=(2, 6, 7), n_text=0, P=3, steps=2, sigma=0.05):
    return Workload(name, B, H, D, tuple(grid), n_text, P, steps, sigma)


def _gen(seed: int, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + int(stream))
    return g


def banded_mask(P: int, width: int = 1) -> np.ndarray:
    """COMPUTE pairs with |i - j| <= width (uint8 [P, P])."""
    i = np.arange(P)
    return (np.abs(i[:, None] - i[None, :]) <= width).astype(np.uint8)


class StepInputs:
    """Iterates the denoising steps of one workload: (q, k, v) bf16 (or fp16) tensors [B, L, H, D]."""

    def __init__(self, wl: Workload, seed: int = 0, device="cpu", dtype=torch.bfloat16):
        self.wl, self.seed, self.device = wl, seed, torch.device(device)
        self.dtype = dtype          # 16-bit type the fp32 masters are rounded to: bfloat16 or float16
        self._masters = None
        self._step = 0

    def _first(self):
        wl, dev = self.wl, self.device
        T, Hg, Wg = wl.grid
        gf = _gen(self.seed, STREAM_FEATURES, "cpu")
        omega = torch.rand(N_FEATURES, 3, generator=gf, dtype=torch.float64) * 0.3
        theta = torch.rand(N_FEATURES, generator=gf, dtype=torch.float64) * (2.0 * math.pi)
        t, h, w = torch.meshgrid(torch.arange(T), torch.arange(Hg), torch.arange(Wg), indexing="ij")
        xyz = torch.stack([t.reshape(-1), h.reshape(-1), w.reshape(-1)], dim=1).to(torch.float64)
        phi = torch.cos(xyz @ omega.T + theta).to(torch.float32).to(dev)          # [Lv, 16]
        a_qk = (torch.randn(wl.H, N_FEATURES, wl.D, generator=_gen(self.seed, STREAM_PROJ_QK, "cpu"))
                * 0.25).to(dev)                                                    # std 1/4 -> variance 1/16
        a_v = (torch.randn(wl.H, N_FEATURES, wl.D, generator=_gen(self.seed, STREAM_PROJ_V, "cpu"))
               * 0.25).to(dev)
        masters = []
        for idx, proj in enumerate((a_qk, a_qk, a_v)):
            g = _gen(self.seed, STREAM_NOISE * 16 + idx, dev)
            x = torch.randn(wl.B, wl.L, wl.H, wl.D, generator=g, device=dev, dtype=torch.float32)
            field_ = torch.einsum("lm,hmd->lhd", phi, proj)                       # [Lv, H, D]
            x[:, wl.n_text:] = 0.6 * x[:, wl.n_text:] + field_.unsqueeze(0)
            masters.append(x)
        return masters

    def next(self):
        wl = self.wl
        if self._masters is None:
            self._masters = self._first()
        else:
            for idx, m in enumerate(self._masters):
                g = _gen(self.seed, (STREAM_STEP * 16 + idx) * 4096 + self._step, self.device)
                m.add_(torch.randn(m.shape, generator=g, device=self.device, dtype=torch.float32),
                       alpha=wl.sigma)
        self._step += 1
        return tuple(m.to(self.dtype) for m in self._masters)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 (or fp16) tensor -> C-contiguous numpy uint16 array of its bit patterns (host)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def sample_rows(wl: Workload, n: int, seed: int = 0, max_heads=None):
    """n seeded (b, h, row) samples, grouped as {(b, h): sorted unique rows}; always includes the
    first and last row of the sequence and rows next to partition boundaries.  max_heads: draw the heads
    from a seeded subset of that many (always containing the first and the last head)."""
    rng = np.random.Generator(np.random.PCG64(seed * 1_000_003 + STREAM_ROWS))
    off = wl.offsets()
    out = {}
    heads = np.arange(wl.H)
    if max_heads is not None and max_heads < wl.H:
        inner = rng.permutation(np.arange(1, wl.H - 1))[:max(0, max_heads - 2)]
        heads = np.unique(np.concatenate([[0, wl.H - 1], inner]))
    special = [0, wl.L - 1] + [int(o) for o in off[1:-1]] + [int(o) - 1 for o in off[1:-1]]
    for s, r in enumerate(special):
        out.setdefault((0, int(heads[s % heads.size])), set()).add(r)
    bs = rng.integers(0, wl.B, size=n)
    hs = heads[rng.integers(0, heads.size, size=n)]
    rs = rng.integers(0, wl.L, size=n)
    for b, h, r in zip(bs, hs, rs):
        out.setdefault((int(b), int(h)), set()).add(int(r))
    return {bh: np.array(sorted(r), dtype=np.int32) for bh, r in sorted(out.items())}
