"""ctypes binding of libditango's C ABI: same names, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch is used for device memory
and streams.  If the shared library is missing this module raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libditango.so")

DT_OK, DT_ERR_INVALID_ARG, DT_ERR_UNSUPPORTED, DT_ERR_STATE, DT_ERR_CUDA, DT_ERR_TIMEOUT, DT_ERR_RANGE = range(7)
DT_STATE_FP32, DT_STATE_BF16 = 0, 1
DT_INPUT_BF16, DT_INPUT_FP16 = 0, 1
DT_MAX_P = 32

EXPORTS = [
    "dt_create", "dt_destroy", "dt_cache_bytes", "dt_bind_cache", "dt_attn_states", "dt_attn_local", "dt_state_merge",
    "dt_compose_reuse", "dt_state_merge_planned", "dt_plan", "dt_plan_grouped", "dt_planner_init", "dt_planner_step", "dt_planner_commit", "dt_planner_get",
    "dt_plan_static", "dt_step_host_workspace_bytes", "dt_step_host", "dt_get_tc", "dt_set_tc",
    "dt_launch_count", "dt_selftest_wait_timeout", "dt_poll", "dt_status_str", "dt_last_error",
    "dt_attn_fused", "dt_num_slots", "dt_slot_ranges", "dt_group_compose", "dt_group_fit", "dt_group_reset",
    "dt_plan_sums", "dt_plan_from_sums",
]


class dt_config(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("L", C.c_int32), ("P", C.c_int32),
                ("part_offsets", C.POINTER(C.c_int32)), ("softmax_scale", C.c_float),
                ("state_dtype", C.c_int32), ("device", C.c_int32), ("group_size", C.c_int32),
                ("input_dtype", C.c_int32)]


class dt_planner_config(C.Structure):
    _fields_ = [("group_size", C.c_int32), ("eps_initial", C.c_double), ("eps_local", C.c_double),
                ("cache_ratio", C.c_double)]


class DitangoError(RuntimeError):
    def __init__(self, status, name, detail=""):
        self.status = status
        super().__init__(f"{name}" + (f": {detail}" if detail else ""))


_lib = None


def lib():
    """Load libditango.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2607_15650_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64p, u8p, f32p, f64p, i32p = (C.c_void_p, C.POINTER(C.c_int64), C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.POINTER(C.c_int32))
    szp = C.POINTER(C.c_size_t)
    sig = {
        "dt_create": (C.c_int, [C.POINTER(vp), C.POINTER(dt_config)]),
        "dt_destroy": (C.c_int, [vp]),
        "dt_cache_bytes": (C.c_int, [C.POINTER(dt_config), szp, szp]),
        "dt_bind_cache": (C.c_int, [vp, vp, f32p, C.c_size_t, C.c_size_t]),
        "dt_attn_states": (C.c_int, [vp, vp, vp, vp, i64p, u8p, C.c_int32, vp]),
        "dt_attn_local": (C.c_int, [vp, vp, vp, vp, i64p, C.c_int32, vp]),
        "dt_state_merge": (C.c_int, [vp, vp, i64p, f32p, vp]),
        "dt_compose_reuse": (C.c_int, [vp, u8p, vp, f32p, vp]),
        "dt_state_merge_planned": (C.c_int, [vp, u8p, vp, f32p, vp, i64p, f32p, vp]),
        "dt_plan": (C.c_int, [vp, C.c_double, C.c_double, u8p, f64p, f64p, vp]),
        "dt_plan_grouped": (C.c_int, [vp, C.c_double, C.c_double, C.c_int32, u8p, f64p, f64p, vp]),
        "dt_plan_sums": (C.c_int, [vp, f64p, vp]),
        "dt_plan_from_sums": (C.c_int, [vp, f64p, C.c_int64, C.c_double, C.c_double, C.c_int32, u8p, f64p, f64p, vp]),
        "dt_planner_init": (C.c_int, [vp, C.POINTER(dt_planner_config), vp, f32p, C.c_size_t, C.c_size_t, vp]),
        "dt_planner_step": (C.c_int, [vp, u8p, vp, f64p, f64p, vp]),
        "dt_planner_commit": (C.c_int, [vp, vp]),
        "dt_planner_get": (C.c_int, [vp, f64p, f64p, f64p, vp]),
        "dt_plan_static": (C.c_int, [f32p, i32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_double,
                           u8p, f64p, f64p, vp]),
        "dt_step_host_workspace_bytes": (C.c_int, [C.POINTER(dt_config), szp]),
        "dt_step_host": (C.c_int, [vp, vp, vp, vp, vp, C.c_int32, vp, vp, vp, C.c_size_t, vp]),
        "dt_get_tc": (C.c_int, [vp, i32p]),
        "dt_set_tc": (C.c_int, [vp, i32p]),
        "dt_launch_count": (C.c_int, [vp, C.POINTER(C.c_uint64)]),
        "dt_selftest_wait_timeout": (C.c_int, [vp, C.c_uint32, vp]),
        "dt_poll": (C.c_int, [vp]),
        "dt_attn_fused": (C.c_int, [vp, vp, vp, vp, i64p, u8p, vp, f32p, vp, i64p, f32p, vp]),
        "dt_num_slots": (C.c_int, [vp, i32p, i32p]),
        "dt_slot_ranges": (C.c_int, [vp, i32p]),
        "dt_group_compose": (C.c_int, [vp, vp]),
        "dt_group_fit": (C.c_int, [vp, C.c_size_t, i32p, vp]),
        "dt_group_reset": (C.c_int, [vp, vp]),
        "dt_status_str": (C.c_char_p, [C.c_int]),
        "dt_last_error": (C.c_char_p, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _lib = L
    return L


def make_config(B, H, D, L, offsets, softmax_scale, state_dtype=DT_STATE_FP32, device=0, group_size=1,
                input_dtype=DT_INPUT_BF16):
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    cfg = dt_config(B, H, D, L, off.size - 1, off.ctypes.data_as(C.POINTER(C.c_int32)), float(softmax_scale),
                    int(state_dtype), int(device), int(group_size), int(input_dtype))
    cfg._keepalive = off
    return cfg


def status_str(s: int) -> str:
    return lib().dt_status_str(int(s)).decode()


def dt_cache_bytes(cfg):
    o, l = C.c_size_t(), C.c_size_t()
    s = lib().dt_cache_bytes(C.byref(cfg), C.byref(o), C.byref(l))
    if s != DT_OK:
        raise DitangoError(s, status_str(s))
    return o.value, l.value


def dt_step_host_workspace_bytes(cfg):
    n = C.c_size_t()
    s = lib().dt_step_host_workspace_bytes(C.byref(cfg), C.byref(n))
    if s != DT_OK:
        raise DitangoError(s, status_str(s))
    return n.value


def _strides4(t: torch.Tensor):
    return (C.c_int64 * 4)(*[int(x) for x in t.stride()])


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


STATIC_PLAN_MAX_PARTIALS = 262144


def dt_plan_static(lse_state, offsets, B, H, L, mask_dev, eps=0.0, target_fraction=-1.0, w_dev=None,
                   eps_out_dev=None, stream=None):
    """Plan without a context and without any allocation inside the library (see ditango.h): for callers
    that may not touch the CUDA allocator when they plan.  `lse_state` is the fp32 LSE cache [P, B, H, L]
    on the device, `offsets` the P+1 partition offsets on the host.  Problems needing more than
    STATIC_PLAN_MAX_PARTIALS partial sums are refused (DT_ERR_UNSUPPORTED)."""
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    P = off.size - 1
    assert lse_state.is_cuda and lse_state.dtype == torch.float32 and lse_state.is_contiguous()
    assert mask_dev.is_cuda and mask_dev.dtype == torch.uint8 and mask_dev.is_contiguous()
    wp = C.c_void_p(w_dev.data_ptr()) if w_dev is not None else C.c_void_p()
    ep = C.c_void_p(eps_out_dev.data_ptr()) if eps_out_dev is not None else C.c_void_p()
    s = lib().dt_plan_static(C.c_void_p(lse_state.data_ptr()), off.ctypes.data_as(C.POINTER(C.c_int32)), int(B), int(H),
                             int(L), int(P), float(eps), float(target_fraction), C.c_void_p(mask_dev.data_ptr()), wp, ep,
                             _stream_ptr(stream))
    if s != DT_OK:
        detail = ("problem exceeds the built-in scratch of %d partial sums" % STATIC_PLAN_MAX_PARTIALS
                  if s == DT_ERR_UNSUPPORTED else "dt_plan_static")
        raise DitangoError(s, status_str(s), detail)


class Context:
    """Owns a dt_ctx and (optionally) the state-cache tensors bound to it."""

    def __init__(self, B, H, D, L, offsets, softmax_scale, state_dtype=DT_STATE_FP32, device=0, alloc_cache=True,
                 group_size=1, input_dtype=DT_INPUT_BF16):
        self._h = C.c_void_p()
        self.cfg = make_config(B, H, D, L, offsets, softmax_scale, state_dtype, device, group_size, input_dtype)
        self.in_dtype = torch.float16 if input_dtype == DT_INPUT_FP16 else torch.bfloat16
        self.device = torch.device("cuda", device)
        s = lib().dt_create(C.byref(self._h), C.byref(self.cfg))
        if s != DT_OK:
            self._h = C.c_void_p()
            raise DitangoError(s, status_str(s), "dt_create")
        self.o_state = self.lse_state = None
        if alloc_cache:
            S = self.dt_num_slots()[0]
            sdt = torch.float32 if state_dtype == DT_STATE_FP32 else torch.bfloat16
            o = torch.empty((S, B, H, L, D), dtype=sdt, device=self.device)
            l = torch.empty((S, B, H, L), dtype=torch.float32, device=self.device)
            self.dt_bind_cache(o, l)

    def _check(self, s):
        if s != DT_OK:
            raise DitangoError(s, status_str(s), lib().dt_last_error(self._h).decode())

    def dt_bind_cache(self, o_state: torch.Tensor, lse_state: torch.Tensor):
        assert o_state.is_cuda and lse_state.is_cuda and o_state.is_contiguous() and lse_state.is_contiguous()
        self._check(lib().dt_bind_cache(self._h, C.c_void_p(o_state.data_ptr()), C.c_void_p(lse_state.data_ptr()),
                                        o_state.numel() * o_state.element_size(), lse_state.numel() * 4))
        self.o_state, self.lse_state = o_state, lse_state

    def dt_attn_states(self, q, k, v, mask_dev, step, stream=None):
        assert q.dtype == k.dtype == v.dtype == self.in_dtype and q.is_cuda
        assert q.stride() == k.stride() == v.stride() and q.shape == k.shape == v.shape
        assert mask_dev.dtype == torch.uint8 and mask_dev.is_cuda and mask_dev.is_contiguous()
        self._check(lib().dt_attn_states(self._h, C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()),
                                         C.c_void_p(v.data_ptr()), _strides4(q), C.c_void_p(mask_dev.data_ptr()),
                                         int(step), _stream_ptr(stream)))

    def dt_attn_local(self, q, k, v, step, stream=None):
        assert q.dtype == k.dtype == v.dtype == self.in_dtype and q.is_cuda
        assert q.stride() == k.stride() == v.stride() and q.shape == k.shape == v.shape
        self._check(lib().dt_attn_local(self._h, C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()),
                                        C.c_void_p(v.data_ptr()), _strides4(q), int(step), _stream_ptr(stream)))

    def dt_attn_fused(self, q, k, v, mask_dev, comp_o, comp_lse, out, lse_out=None, stream=None):
        assert q.dtype == k.dtype == v.dtype == self.in_dtype and q.is_cuda
        assert q.stride() == k.stride() == v.stride() and q.shape == k.shape == v.shape
        assert mask_dev.dtype == torch.uint8 and mask_dev.is_cuda and mask_dev.is_contiguous()
        assert out.dtype == self.in_dtype and out.is_cuda
        opt = lambda t: C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p()
        if comp_o is not None and comp_lse is not None:
            assert comp_o.is_contiguous() and comp_lse.is_contiguous() and comp_o.dtype == self.o_state.dtype
        self._check(lib().dt_attn_fused(self._h, C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                        _strides4(q), C.c_void_p(mask_dev.data_ptr()), opt(comp_o), opt(comp_lse),
                                        C.c_void_p(out.data_ptr()), _strides4(out), opt(lse_out), _stream_ptr(stream)))

    def dt_state_merge(self, out, lse_out=None, stream=None):
        assert out.dtype == self.in_dtype and out.is_cuda
        lp = C.c_void_p(lse_out.data_ptr()) if lse_out is not None else C.c_void_p()
        if lse_out is not None:
            assert lse_out.dtype == torch.float32 and lse_out.is_contiguous()
        self._check(lib().dt_state_merge(self._h, C.c_void_p(out.data_ptr()), _strides4(out), lp, _stream_ptr(stream)))

    def dt_compose_reuse(self, mask_dev, comp_o, comp_lse, stream=None):
        assert comp_o.is_cuda and comp_o.is_contiguous() and comp_o.dtype == self.o_state.dtype
        assert comp_lse.is_cuda and comp_lse.is_contiguous() and comp_lse.dtype == torch.float32
        self._check(lib().dt_compose_reuse(self._h, C.c_void_p(mask_dev.data_ptr()), C.c_void_p(comp_o.data_ptr()),
                                           C.c_void_p(comp_lse.data_ptr()), _stream_ptr(stream)))

    def dt_state_merge_planned(self, mask_dev, comp_o, comp_lse, out, lse_out=None, stream=None):
        assert out.dtype == self.in_dtype and out.is_cuda
        lp = C.c_void_p(lse_out.data_ptr()) if lse_out is not None else C.c_void_p()
        self._check(lib().dt_state_merge_planned(self._h, C.c_void_p(mask_dev.data_ptr()), C.c_void_p(comp_o.data_ptr()),
                                                 C.c_void_p(comp_lse.data_ptr()), C.c_void_p(out.data_ptr()),
                                                 _strides4(out), lp, _stream_ptr(stream)))

    def dt_planner_init(self, snap_o, snap_lse, group_size=1, eps_initial=0.0, eps_local=0.1, cache_ratio=0.5, stream=None):
        assert snap_o.is_cuda and snap_o.is_contiguous() and snap_o.dtype == self.o_state.dtype
        assert snap_lse.is_cuda and snap_lse.is_contiguous() and snap_lse.dtype == torch.float32
        pc = dt_planner_config(int(group_size), float(eps_initial), float(eps_local), float(cache_ratio))
        self._check(lib().dt_planner_init(self._h, C.byref(pc), C.c_void_p(snap_o.data_ptr()), C.c_void_p(snap_lse.data_ptr()),
                                          snap_o.numel() * snap_o.element_size(), snap_lse.numel() * 4, _stream_ptr(stream)))
        self._snap = (snap_o, snap_lse)

    def dt_planner_step(self, mask_dev, is_anchor_dev=None, ase_dev=None, delta_rel_dev=None, stream=None):
        opt = lambda t: C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p()
        self._check(lib().dt_planner_step(self._h, C.c_void_p(mask_dev.data_ptr()), opt(is_anchor_dev), opt(ase_dev),
                                          opt(delta_rel_dev), _stream_ptr(stream)))

    def dt_planner_commit(self, stream=None):
        self._check(lib().dt_planner_commit(self._h, _stream_ptr(stream)))

    def dt_planner_get(self):
        P, S = self.cfg.P, self.dt_num_slots()[0]
        w = np.empty((P, S), dtype=np.float64); alpha = np.empty((P, S), dtype=np.float64)
        eps = C.c_double(); have = C.c_int32()
        self._check(lib().dt_planner_get(self._h, w.ctypes.data_as(C.c_void_p), alpha.ctypes.data_as(C.c_void_p),
                                         C.byref(eps), C.byref(have)))
        return w, alpha, eps.value, bool(have.value)

    def dt_plan_grouped(self, mask_dev, group_size, eps=0.0, target_fraction=-1.0, w_dev=None, eps_out_dev=None,
                        stream=None):
        wp = C.c_void_p(w_dev.data_ptr()) if w_dev is not None else C.c_void_p()
        ep = C.c_void_p(eps_out_dev.data_ptr()) if eps_out_dev is not None else C.c_void_p()
        self._check(lib().dt_plan_grouped(self._h, float(eps), float(target_fraction), int(group_size),
                                          C.c_void_p(mask_dev.data_ptr()), wp, ep, _stream_ptr(stream)))

    def dt_plan_sums(self, sums_dev, stream=None):
        assert sums_dev.dtype == torch.float64 and sums_dev.is_cuda and sums_dev.is_contiguous()
        self._check(lib().dt_plan_sums(self._h, C.c_void_p(sums_dev.data_ptr()), _stream_ptr(stream)))

    def dt_plan_from_sums(self, sums_dev, total_bh, mask_dev, eps=0.0, target_fraction=-1.0, group_size=1, w_dev=None,
                          eps_out_dev=None, stream=None):
        assert sums_dev.dtype == torch.float64 and sums_dev.is_cuda and sums_dev.is_contiguous()
        assert mask_dev.dtype == torch.uint8 and mask_dev.is_cuda and mask_dev.is_contiguous()
        wp = C.c_void_p(w_dev.data_ptr()) if w_dev is not None else C.c_void_p()
        ep = C.c_void_p(eps_out_dev.data_ptr()) if eps_out_dev is not None else C.c_void_p()
        self._check(lib().dt_plan_from_sums(self._h, C.c_void_p(sums_dev.data_ptr()), int(total_bh), float(eps),
                                            float(target_fraction), int(group_size), C.c_void_p(mask_dev.data_ptr()),
                                            wp, ep, _stream_ptr(stream)))

    def dt_plan(self, mask_dev, eps=0.0, target_fraction=-1.0, w_dev=None, eps_out_dev=None, stream=None):
        assert mask_dev.dtype == torch.uint8 and mask_dev.is_cuda and mask_dev.is_contiguous()
        wp = C.c_void_p(w_dev.data_ptr()) if w_dev is not None else C.c_void_p()
        ep = C.c_void_p(eps_out_dev.data_ptr()) if eps_out_dev is not None else C.c_void_p()
        if w_dev is not None:
            assert w_dev.dtype == torch.float64 and w_dev.is_contiguous()
        if eps_out_dev is not None:
            assert eps_out_dev.dtype == torch.float64
        self._check(lib().dt_plan(self._h, float(eps), float(target_fraction), C.c_void_p(mask_dev.data_ptr()), wp, ep,
                                  _stream_ptr(stream)))

    def dt_step_host(self, q_host, k_host, v_host, mask_host, step, out_host, lse_out_host, workspace, stream=None):
        lp = C.c_void_p(lse_out_host.data_ptr()) if lse_out_host is not None else C.c_void_p()
        self._check(lib().dt_step_host(self._h, C.c_void_p(q_host.data_ptr()), C.c_void_p(k_host.data_ptr()),
                                       C.c_void_p(v_host.data_ptr()), C.c_void_p(mask_host.data_ptr()), int(step),
                                       C.c_void_p(out_host.data_ptr()), lp, C.c_void_p(workspace.data_ptr()),
                                       workspace.numel() * workspace.element_size(), _stream_ptr(stream)))

    def dt_num_slots(self):
        """(cache slots S, current group size g)."""
        S, g = C.c_int32(), C.c_int32()
        self._check(lib().dt_num_slots(self._h, C.byref(S), C.byref(g)))
        return int(S.value), int(g.value)

    def dt_slot_ranges(self):
        """int32 [P, S, 4]: keys [r1, r1+n1) and [r2, r2+n2) of every (query partition, slot)."""
        S = self.dt_num_slots()[0]
        r = np.empty((self.cfg.P, S, 4), dtype=np.int32)
        self._check(lib().dt_slot_ranges(self._h, r.ctypes.data_as(C.POINTER(C.c_int32))))
        return r

    def dt_group_compose(self, stream=None):
        self._check(lib().dt_group_compose(self._h, _stream_ptr(stream)))

    def dt_group_fit(self, max_bytes, stream=None) -> int:
        """Compose groups (Eq. 15) until the slots in use fit into max_bytes; returns how many compositions ran."""
        n = C.c_int32()
        self._check(lib().dt_group_fit(self._h, int(max_bytes), C.byref(n), _stream_ptr(stream)))
        return int(n.value)

    def dt_group_reset(self, stream=None):
        self._check(lib().dt_group_reset(self._h, _stream_ptr(stream)))

    def dt_get_tc(self):
        P = self.cfg.P
        tc = np.empty((P, self.dt_num_slots()[0]), dtype=np.int32)
        self._check(lib().dt_get_tc(self._h, tc.ctypes.data_as(C.POINTER(C.c_int32))))
        return tc

    def dt_set_tc(self, tc):
        tc = np.ascontiguousarray(tc, dtype=np.int32)
        self._check(lib().dt_set_tc(self._h, tc.ctypes.data_as(C.POINTER(C.c_int32))))

    def dt_launch_count(self) -> int:
        n = C.c_uint64()
        self._check(lib().dt_launch_count(self._h, C.byref(n)))
        return int(n.value)

    def dt_selftest_wait_timeout(self, limit_us=1000, stream=None):
        self._check(lib().dt_selftest_wait_timeout(self._h, int(limit_us), _stream_ptr(stream)))

    def dt_poll(self):
        """Raises DitangoError if the device recorded a condition; returns None otherwise."""
        self._check(lib().dt_poll(self._h))

    def close(self):
        if self._h:
            lib().dt_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
