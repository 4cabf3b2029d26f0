"""Host-only checks of the C-ABI library: it loads, exports every symbol the header declares, and
its closed-form / argument-checking entry points behave (no kernel launch, no GPU needed)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2607_15650_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ditango.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dt_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_cache_bytes_closed_form_and_half_of_kv(lib):
    """State size accounting: per pair OUT (n_i H D) + LSE (n_i H) against 2 n_j H D of KV --
    'half of KV size' when the state is stored in the KV dtype (Section 2.2.4)."""
    wl = inputs.WORKLOADS["c3_wan720p"]
    for sdt, eb in ((binding.DT_STATE_FP32, 4), (binding.DT_STATE_BF16, 2)):
        cfg = binding.make_config(wl.B, wl.H, wl.D, wl.L, wl.offsets(), wl.scale, sdt)
        o, l = binding.dt_cache_bytes(cfg)
        assert o == wl.P * wl.B * wl.H * wl.L * wl.D * eb
        assert l == wl.P * wl.B * wl.H * wl.L * 4
    kv_bytes_per_pair = 2 * 4725 * wl.H * wl.D * 2
    state_bytes_per_pair = 4725 * wl.H * wl.D * 2
    assert state_bytes_per_pair * 2 == kv_bytes_per_pair
    ws = binding.dt_step_host_workspace_bytes(cfg)
    assert ws >= 4 * wl.L * wl.H * wl.D * 2 + wl.L * wl.H * 4


@pytest.mark.parametrize("kw,status", [
    (dict(D=96), binding.DT_ERR_UNSUPPORTED),
    (dict(P=33), binding.DT_ERR_UNSUPPORTED),
    (dict(state_dtype=7), binding.DT_ERR_UNSUPPORTED),
    (dict(scale=0.0), binding.DT_ERR_INVALID_ARG),
    (dict(offsets=[0, 5, 5, 12]), binding.DT_ERR_INVALID_ARG),
    (dict(offsets=[1, 5, 8, 12]), binding.DT_ERR_INVALID_ARG),
    (dict(offsets=[0, 5, 8, 11]), binding.DT_ERR_INVALID_ARG),
])
def test_bad_configs_are_rejected_before_any_cuda_call(lib, kw, status):
    P = kw.get("P", 3)
    offsets = kw.get("offsets", np.linspace(0, 12 * P, P + 1).astype(int) if P != 3 else [0, 4, 8, 12])
    L = 12 if P == 3 else 12 * P
    cfg = binding.make_config(1, 2, kw.get("D", 64), L, offsets, kw.get("scale", 0.125), kw.get("state_dtype", 0))
    o, l = C.c_size_t(), C.c_size_t()
    assert lib.dt_cache_bytes(C.byref(cfg), C.byref(o), C.byref(l)) == status
    h = C.c_void_p()
    assert lib.dt_create(C.byref(h), C.byref(cfg)) == status
    assert not h


def test_status_strings(lib):
    assert binding.status_str(0) == "DT_OK"
    assert binding.status_str(binding.DT_ERR_STATE) == "DT_ERR_STATE"
    assert binding.status_str(99) == "DT_ERR_UNKNOWN"
    assert lib.dt_destroy(None) == binding.DT_OK
    assert lib.dt_poll(None) == binding.DT_ERR_INVALID_ARG


def test_null_context_is_an_argument_error_on_every_entry_point(lib):
    """Every call that takes a context returns DT_ERR_INVALID_ARG for a null one (dt_destroy accepts it, like free);
    nothing is dereferenced and no CUDA call is made."""
    text = open(os.path.join(ROOT, "include", "ditango.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    with_ctx = sorted(set(re.findall(r"\bdt_status\s+(dt_[a-z_0-9]+)\s*\(\s*dt_ctx\s*\*\s*ctx\b", text)))
    assert len(with_ctx) >= 25 and "dt_plan" in with_ctx and "dt_plan_grouped" in with_ctx
    for name in with_ctx:
        fn = getattr(lib, name)
        args = []
        for t in fn.argtypes[1:]:
            if t in (C.c_double, C.c_float):
                args.append(0.0)
            elif t in (C.c_int32, C.c_int64, C.c_uint32, C.c_size_t, C.c_int):
                args.append(0)
            else:
                args.append(None)
        got = fn(None, *args)
        assert got == (binding.DT_OK if name == "dt_destroy" else binding.DT_ERR_INVALID_ARG), name
    assert lib.dt_last_error(None) in (b"", None) or isinstance(lib.dt_last_error(None), bytes)
