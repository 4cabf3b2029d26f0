"""Seeded random configurations of the whole path (partition counts and sizes, head sizes, batch, cache and input
types, group sizes, masks), every state and every merged output against the oracle.  Small sizes, many shapes:
meant to catch index arithmetic that the hand-picked cases miss."""
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs
from tests.test_gpu_fused import _fused_steps
from tests.test_gpu_groups import GroupRun
from tests.test_gpu_parity import Run

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def _random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    B = int(rng.choice([1, 1, 2]))
    H = int(rng.integers(1, 4))
    P = int(rng.integers(1, 9))
    grid = (int(rng.integers(1, 5)), int(rng.integers(5, 21)), int(rng.integers(5, 21)))     # up to 1600 tokens
    n_text = int(rng.choice([0, 0, 3, 17]))
    L = n_text + grid[0] * grid[1] * grid[2]
    P = min(P, L // 2)
    cuts = np.sort(rng.choice(np.arange(1, L), size=P - 1, replace=False)) if P > 1 else np.array([], dtype=np.int64)
    offsets = [0] + [int(c) for c in cuts] + [L]
    g = int(rng.choice([1, 1, 2, 3, 4]))
    g = 1 if P == 1 else min(g, P)
    state_dtype = int(rng.choice([binding.DT_STATE_FP32, binding.DT_STATE_BF16]))
    fp16 = bool(rng.integers(0, 2))
    return rng, D, B, H, P, grid, n_text, offsets, g, state_dtype, fp16


# DT_FUZZ_CASES / DT_FUZZ_FIRST: how many seeds and the first one (a longer soak takes a later range)
_FIRST = int(os.environ.get("DT_FUZZ_FIRST", "0"))


@pytest.mark.parametrize("seed", range(_FIRST, _FIRST + int(os.environ.get("DT_FUZZ_CASES", "24"))))
def test_random_configuration(seed):
    rng, D, B, H, P, grid, n_text, offsets, g, state_dtype, fp16 = _random_case(seed)
    wl = inputs.Workload(f"fuzz{seed}", B, H, D, grid, n_text, P, 3, 0.05)
    assert wl.L == offsets[-1]
    if g > 1:
        run = GroupRun(wl, g, offsets=offsets, seed=seed, state_dtype=state_dtype, fp16=fp16)
        S, local_col = run.S, (lambda i: 0)
    else:
        run = Run(wl, offsets=offsets, seed=seed, state_dtype=state_dtype, fp16=fp16)
        S, local_col = P, (lambda i: i)

    def random_mask(p_compute):
        m = (rng.random((P, S)) < p_compute).astype(np.uint8)
        for i in range(P):
            m[i, local_col(i)] = 1
        return m

    run.step(np.ones((P, S), np.uint8), check_states=True)
    run.step(random_mask(0.5), check_states=True)
    run.step(random_mask(0.2), check_states=True)
    if seed % 3 == 0:
        # the fused pass on the same context: its own anchor step, then two masks
        sdt = torch.float32 if state_dtype == binding.DT_STATE_FP32 else torch.bfloat16
        _fused_steps(run, P, S, [random_mask(0.5), random_mask(0.0)], state_dtype=sdt)
    if g > 1 and seed % 2 == 0 and run.S - 1 >= 2:
        run.ctx.dt_group_compose()
        run.ses.compose()
        if state_dtype == binding.DT_STATE_BF16:
            run.tol_scale = 2.0          # composed states have been rounded to bf16 twice
        run.check_layout()
        torch.cuda.synchronize()
        run.check_states("after compose")
        S2 = run.S
        m = np.zeros((P, S2), np.uint8); m[:, 0] = 1; m[::2, S2 - 1] = 1
        run.step(m, check_states=True)
