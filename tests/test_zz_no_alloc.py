"""dt_plan_static -- the plan entry point for callers that cannot allocate device memory -- against
dt_plan on the same LSE cache, through the C ABI, twice in a row.

Such callers exist: a serving process that carved its memory pools at start-up and forbids
cudaMalloc afterwards, or code on a path where touching the allocator is not allowed.  The
allocation-free variant keeps its partial sums in an array inside the library image, shared by
every call, so the second call runs on whatever the first one left there; this file checks that
both calls still agree with the context-based entry point bit for bit, and that an oversized
problem is refused.  It sorts last so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build

pytestmark = pytest.mark.gpu


def _case(rng, B, H, L, off, dev):
    P = len(off) - 1
    part = np.searchsorted(off, np.arange(L), side="right") - 1
    dist = np.abs(np.subtract.outer(np.arange(P), np.arange(P)))
    lse = rng.standard_normal((P, B, H, L)) * 0.7
    for j in range(P):
        lse[j] -= 0.9 * dist[part, j]
    return torch.from_numpy(lse.astype(np.float32)).to(dev)


def _both(lse, off, B, H, L, D, dev, **kw):
    P = len(off) - 1
    ctx = binding.Context(B, H, D, L, off, 0.1, alloc_cache=False)
    ctx.dt_bind_cache(torch.empty((P, B, H, L, D), device=dev), lse)
    outs = []
    for fn in ("ctx", "static"):
        mask = torch.zeros(P * P, dtype=torch.uint8, device=dev)
        W = torch.zeros(P * P, dtype=torch.float64, device=dev)
        eps = torch.zeros(1, dtype=torch.float64, device=dev)
        if fn == "ctx":
            ctx.dt_plan(mask, w_dev=W, eps_out_dev=eps, **kw)
        else:
            free0 = torch.cuda.mem_get_info()[0]
            binding.dt_plan_static(lse, off, B, H, L, mask, w_dev=W, eps_out_dev=eps, **kw)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0          # the call took no device memory
        torch.cuda.synchronize()
        outs.append((mask.cpu().numpy(), W.cpu().numpy(), eps.item()))
    return outs


def test_static_plan_matches_context_plan_on_two_calls_in_a_row():
    build.build()
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(21)
    # first call: the larger problem
    off1 = np.array([0, 1500, 2900, 4100, 6000], np.int32)
    lse1 = _case(rng, 2, 3, 6000, off1, dev)
    (m_a, w_a, e_a), (m_b, w_b, e_b) = _both(lse1, off1, 2, 3, 6000, 64, dev, target_fraction=0.5)
    assert (m_a == m_b).all() and m_a.sum() == 8
    assert (w_b == w_a).all() and e_b == e_a               # the same kernels in the same order: bit for bit
    np.testing.assert_allclose(w_b.reshape(4, 4).sum(1), 1.0, atol=1e-5)
    # and against the oracle: its measure from the same fp32 LSEs, its rule on the device's own W
    W_ref = orc.contribution(lse1.cpu().numpy().astype(np.float64), off1)
    np.testing.assert_allclose(w_b.reshape(4, 4), W_ref, rtol=2e-5, atol=1e-10)
    own_mask, own_eps, _ = orc.target_fraction(w_b.reshape(4, 4), 0.5)
    assert (m_b.reshape(4, 4) == own_mask).all() and e_b == own_eps
    ref_mask, ref_eps, _ = orc.target_fraction(W_ref, 0.5)
    if (np.abs(W_ref - ref_eps)[~np.eye(4, dtype=bool)].min() / ref_eps) > 1e-4:
        assert (m_b.reshape(4, 4) == ref_mask).all()
    # second call: a smaller, differently partitioned problem on top of the first call's leftovers
    off2 = np.array([0, 40, 300, 301, 777], np.int32)
    lse2 = _case(rng, 1, 2, 777, off2, dev)
    (m_a, w_a, e_a), (m_b, w_b, e_b) = _both(lse2, off2, 1, 2, 777, 64, dev, eps=0.12)
    assert (m_a == m_b).all() and (w_b == w_a).all()
    assert e_b == e_a == 0.12
    assert (m_b.reshape(4, 4) == orc.threshold(w_b.reshape(4, 4), 0.12)).all()
    np.testing.assert_allclose(w_b.reshape(4, 4), orc.contribution(lse2.cpu().numpy().astype(np.float64), off2), rtol=2e-5, atol=1e-10)


def test_static_plan_accepts_exactly_its_limit_and_refuses_one_step_beyond():
    """262 144 partial sums fit: B*H = 256 with P = 32 and one chunk of rows is exactly that and runs (target mode, no W
    asked for); one more head is refused before anything is launched."""
    build.build()
    dev = torch.device("cuda", 0)
    P, B, L = 32, 1, 64
    off = np.arange(0, L + 1, 2, dtype=np.int32)
    for H, fits in ((256, True), (257, False)):
        lse = torch.zeros((P, B, H, L), dtype=torch.float32, device=dev)
        mask = torch.full((P * P,), 7, dtype=torch.uint8, device=dev)
        if fits:
            binding.dt_plan_static(lse, off, B, H, L, mask, target_fraction=0.25)
            torch.cuda.synchronize()
            got = mask.cpu().numpy().reshape(P, P)
            assert got.sum() == 256 and (np.diag(got) == 1).all()        # K = round(0.25 * 1024), diagonal forced
        else:
            with pytest.raises(binding.DitangoError) as ei:
                binding.dt_plan_static(lse, off, B, H, L, mask, target_fraction=0.25)
            assert ei.value.status == binding.DT_ERR_UNSUPPORTED
            torch.cuda.synchronize()
            assert (mask == 7).all()


def test_static_plan_refuses_problems_beyond_its_scratch():
    build.build()
    dev = torch.device("cuda", 0)
    P, B, H = 32, 1, 300                                    # 300 * 32 * 32 * 1 = 307200 > 262144
    L = 64
    off = np.arange(0, L + 1, 2, dtype=np.int32)
    lse = torch.zeros((P, B, H, L), dtype=torch.float32, device=dev)
    mask = torch.full((P * P,), 7, dtype=torch.uint8, device=dev)
    with pytest.raises(binding.DitangoError) as ei:
        binding.dt_plan_static(lse, off, B, H, L, mask, eps=0.1)
    assert ei.value.status == binding.DT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert (mask == 7).all()                                # refused before anything ran
