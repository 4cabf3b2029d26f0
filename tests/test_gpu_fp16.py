"""GPU parity with FP16 inputs (Table 1: the Wan models run in FP16): q, k, v and the attention output are
fp16, P is rounded to fp16 for the PV product, accumulation and the state cache are as for bf16.  Same
tolerances as for bf16 (fp16 carries three more mantissa bits)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_15650_b200 import binding, build, inputs
from tests.test_gpu_fused import _fused_steps
from tests.test_gpu_groups import GroupRun
from tests.test_gpu_parity import Run, check_lse, check_o

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def test_fp16_config0_two_steps():
    wl = inputs.WORKLOADS["c0_correctness"]
    run = Run(wl, fp16=True)
    run.step(np.ones((4, 4), np.uint8), check_states=True)
    run.step(inputs.banded_mask(4, 1), check_states=True)


@pytest.mark.parametrize("state_dtype", [binding.DT_STATE_FP32, binding.DT_STATE_BF16])
def test_fp16_d128_ragged_with_text_rows(state_dtype):
    wl = inputs.Workload("fp16_ragged", 2, 2, 128, (3, 9, 11), 5, 3, 2, 0.05)
    run = Run(wl, offsets=[0, 100, 230, 302], seed=3, fp16=True, state_dtype=state_dtype)
    run.step(np.ones((3, 3), np.uint8), check_states=True)
    run.step(np.eye(3, dtype=np.uint8), check_states=True)


def test_fp16_grouped_cache_and_fused_pass():
    wl = inputs.Workload("fp16_groups", 1, 2, 128, (4, 10, 12), 0, 6, 3, 0.05)
    run = GroupRun(wl, 2, seed=5, fp16=True)
    S = run.S
    local = np.zeros((6, S), np.uint8); local[:, 0] = 1
    some = local.copy(); some[:, 2] = 1
    _fused_steps(run, 6, S, [some, local])


def test_fp16_host_step_and_dtype_checks():
    wl = inputs.Workload("fp16_host", 1, 4, 64, (2, 8, 9), 0, 2, 1, 0.05)
    dev = torch.device("cuda", 0)
    ctx = binding.Context(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale, input_dtype=binding.DT_INPUT_FP16)
    q, k, v = inputs.StepInputs(wl, seed=1, device="cpu", dtype=torch.float16).next()
    qh, kh, vh = (x.pin_memory() for x in (q, k, v))
    oh = torch.empty((wl.B, wl.L, wl.H, wl.D), dtype=torch.float16).pin_memory()
    lh = torch.empty((wl.B, wl.H, wl.L), dtype=torch.float32).pin_memory()
    ws = torch.empty(binding.dt_step_host_workspace_bytes(ctx.cfg), dtype=torch.uint8, device=dev)
    ctx.dt_step_host(qh, kh, vh, torch.ones(4, dtype=torch.uint8), 0, oh, lh, ws)
    ctx.dt_poll()
    qb, kb, vb = (inputs.bf16_bits(x) for x in (q, k, v))
    for h in range(wl.H):
        ro, rl = orc.full_attention(qb, kb, vb, wl.scale, 0, h, np.arange(wl.L, dtype=np.int32), fp16=True)
        check_o(oh[0, :, h].float().numpy(), ro, "fp16 host step")
        check_lse(lh[0, h].numpy(), rl, "fp16 host step")
    with pytest.raises(AssertionError):          # a bf16 tensor on an fp16 context is refused by the binding
        ctx.dt_attn_states(q.to(dev).to(torch.bfloat16), k.to(dev).to(torch.bfloat16), v.to(dev).to(torch.bfloat16),
                           torch.ones(4, dtype=torch.uint8, device=dev), 1)
    bad = binding.make_config(1, 1, 64, 128, [0, 128], 0.125, input_dtype=7)
    h = binding.C.c_void_p()
    assert binding.lib().dt_create(binding.C.byref(h), binding.C.byref(bad)) == binding.DT_ERR_UNSUPPORTED
