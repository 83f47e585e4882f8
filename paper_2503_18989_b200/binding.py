"""Thin ctypes binding of the C-ABI library declared in include/hat.h.

Argument marshalling only: every step of the path runs in the CUDA library.
Functions carry the same names as the C entry points; each raises HatError on a
non-zero status.  There is no fallback: if libhat.so has not been built,
loading raises immediately.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# HAT_LIB=debug loads the build with device-side index checks (python -m paper_2503_18989_b200.build --debug)
LIB_PATH = os.path.join(_HERE, "libhat_debug.so" if os.environ.get("HAT_LIB") == "debug" else "libhat.so")

HAT_OK = 0
HAT_ERR_INVALID_ARG = -1
HAT_ERR_UNSUPPORTED = -2
HAT_ERR_OUT_OF_RANGE = -3
HAT_ERR_WORKSPACE_TOO_SMALL = -4
HAT_ERR_CUDA = -5
HAT_ERR_DEVICE_TIMEOUT = -6
HAT_ERR_TOO_LARGE = -7
HAT_ERR_DEVICE_BOUNDS = -8
HAT_DTYPE_FP16 = 0
HAT_DTYPE_BF16 = 1
HAT_PLAN_HOST_ONLY = 1
DTYPE_CODE = {"fp16": HAT_DTYPE_FP16, "bf16": HAT_DTYPE_BF16}

EXPORTS = [
    "hat_status_string", "hat_version", "hat_last_cuda_error", "hat_launch_count",
    "hat_plan_create", "hat_plan_get_info", "hat_plan_workspace_bytes", "hat_plan_destroy",
    "hat_kv_append", "hat_kv_append_rope", "hat_rope_q", "hat_qkv_rope_append", "hat_chunk_attention", "hat_chunk_attention_out16",
    "hat_plan_staging_bytes",
    "hat_chunk_attention_host",
    "hat_last_device_status", "hat_plan_enable_timing", "hat_plan_read_timing",
    "hat_verify_attention_static", "hat_static_key_range", "hat_plan_set_wait_limit",
    "hat_plan_verify_event", "hat_plan_wait_verify",
    "hat_ctrl_create", "hat_ctrl_destroy", "hat_ctrl_observe", "hat_ctrl_mu", "hat_ctrl_predict",
    "hat_ctrl_device_observe", "hat_ctrl_device_state", "hat_ctrl_chunk_size", "hat_ctrl_parallel_draft_steps",
]
HAT_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024
HAT_STATIC_SPLITS = 8
HAT_TIMING_SLOTS = 4


class hat_cache_desc(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("dtype", C.c_int32), ("num_pages", C.c_int32),
                ("page_size", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("reserved", C.c_int32), ("stride_page", C.c_int64), ("stride_token", C.c_int64),
                ("stride_head", C.c_int64)]


class hat_batch_desc(C.Structure):
    _fields_ = [("num_requests", C.c_int32), ("num_q_heads", C.c_int32), ("max_pages", C.c_int32),
                ("flags", C.c_uint32), ("cu_chunk", C.c_void_p), ("prefix_len", C.c_void_p),
                ("chunk_len", C.c_void_p), ("block_table", C.c_void_p), ("tree_mask", C.c_void_p)]


class hat_plan_info(C.Structure):
    _fields_ = [("num_requests", C.c_int32), ("total_rows", C.c_int32), ("num_verify_requests", C.c_int32),
                ("num_prefill_requests", C.c_int32), ("num_verify_items", C.c_int32),
                ("num_prefill_items", C.c_int32), ("num_merge_rows", C.c_int32), ("max_splits", C.c_int32),
                ("verify_split_len", C.c_int32), ("prefill_split_len", C.c_int32),
                ("prefill_tile_rows", C.c_int32), ("prefill_kernel", C.c_int32),
                ("workspace_bytes", C.c_int64), ("attn_flops", C.c_int64), ("kv_read_bytes", C.c_int64),
                ("stream_kernel", C.c_int32), ("reserved", C.c_int32)]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class HatError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = f"{where}: status {status} ({hat_status_string(status)})"
        if status == HAT_ERR_CUDA:
            msg += f", cudaError {hat_last_cuda_error()}"
        super().__init__(msg)


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Load libhat.so (built by paper_2503_18989_b200.build); fails loudly if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_18989_b200.build` "
                               "(there is no non-CUDA path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
        L.hat_status_string.restype = C.c_char_p
        L.hat_status_string.argtypes = [i32]
        L.hat_version.restype = i32
        L.hat_version.argtypes = []
        L.hat_last_cuda_error.restype = i32
        L.hat_last_cuda_error.argtypes = []
        L.hat_launch_count.restype = C.c_int64
        L.hat_launch_count.argtypes = []
        L.hat_plan_create.restype = i32
        L.hat_plan_create.argtypes = [C.POINTER(hat_cache_desc), C.POINTER(hat_batch_desc), C.POINTER(vp)]
        L.hat_plan_get_info.restype = i32
        L.hat_plan_get_info.argtypes = [vp, C.POINTER(hat_plan_info)]
        L.hat_plan_workspace_bytes.restype = i32
        L.hat_plan_workspace_bytes.argtypes = [vp, C.POINTER(sz)]
        L.hat_plan_destroy.restype = i32
        L.hat_plan_destroy.argtypes = [vp]
        L.hat_kv_append.restype = i32
        L.hat_kv_append.argtypes = [C.POINTER(hat_cache_desc), vp, vp, vp, vp]
        L.hat_kv_append_rope.restype = i32
        L.hat_kv_append_rope.argtypes = [C.POINTER(hat_cache_desc), vp, vp, vp, C.c_float, i32, vp]
        L.hat_rope_q.restype = i32
        L.hat_rope_q.argtypes = [vp, vp, vp, C.c_float, i32, vp]
        L.hat_qkv_rope_append.restype = i32
        L.hat_qkv_rope_append.argtypes = [C.POINTER(hat_cache_desc), vp, vp, i32, vp, vp, C.c_float, i32, vp]
        L.hat_chunk_attention.restype = i32
        L.hat_chunk_attention.argtypes = [C.POINTER(hat_cache_desc), vp, vp, vp, vp, vp, vp, C.c_float, vp, sz, vp]
        L.hat_chunk_attention_out16.restype = i32
        L.hat_chunk_attention_out16.argtypes = [C.POINTER(hat_cache_desc), vp, vp, vp, vp, vp, vp, C.c_float, vp, sz, vp]
        L.hat_plan_staging_bytes.restype = i32
        L.hat_plan_staging_bytes.argtypes = [vp, C.POINTER(sz)]
        L.hat_chunk_attention_host.restype = i32
        L.hat_chunk_attention_host.argtypes = [C.POINTER(hat_cache_desc), vp, vp, vp, vp, vp, vp, C.c_float,
                                               vp, sz, vp, sz, vp]
        L.hat_last_device_status.restype = i32
        L.hat_last_device_status.argtypes = [vp, vp, C.POINTER(i32)]
        L.hat_plan_enable_timing.restype = i32
        L.hat_plan_enable_timing.argtypes = [vp, i32]
        L.hat_plan_read_timing.restype = i32
        L.hat_plan_read_timing.argtypes = [vp, vp, i32, C.POINTER(i32)]
        L.hat_plan_set_wait_limit.restype = i32
        L.hat_plan_set_wait_limit.argtypes = [vp, C.c_longlong, i32]
        dbl = C.c_double
        for name, args in (("hat_ctrl_create", [dbl, dbl, i32, i32, C.POINTER(vp)]), ("hat_ctrl_destroy", [vp]),
                           ("hat_ctrl_observe", [vp, dbl, dbl]), ("hat_ctrl_mu", [vp, C.POINTER(dbl)]),
                           ("hat_ctrl_predict", [vp, dbl, C.POINTER(dbl)]),
                           ("hat_ctrl_device_observe", [vp, i32, dbl, dbl, dbl]),
                           ("hat_ctrl_device_state", [vp, i32, C.POINTER(dbl), C.POINTER(dbl), C.POINTER(dbl)]),
                           ("hat_ctrl_chunk_size", [vp, i32, dbl, i32, i32, i32, C.POINTER(i32)]),
                           ("hat_ctrl_parallel_draft_steps", [vp, i32, i32, dbl, C.POINTER(i32)])):
            getattr(L, name).restype = i32
            getattr(L, name).argtypes = args
        L.hat_plan_verify_event.restype = i32
        L.hat_plan_verify_event.argtypes = [vp, C.POINTER(vp)]
        L.hat_plan_wait_verify.restype = i32
        L.hat_plan_wait_verify.argtypes = [vp]
        L.hat_verify_attention_static.restype = i32
        L.hat_verify_attention_static.argtypes = [C.POINTER(hat_cache_desc), i32, i32, i32, i32, vp, vp, vp, vp,
                                                  vp, vp, vp, C.c_float, vp]
        L.hat_static_key_range.restype = i32
        L.hat_static_key_range.argtypes = [i32, i32, i32, i32, i32] + [C.POINTER(i32)] * 4
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != HAT_OK:
        raise HatError(status, where)


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return int(x.data_ptr())


def hat_status_string(status: int) -> str:
    return lib().hat_status_string(int(status)).decode()


def hat_version() -> int:
    return int(lib().hat_version())


def hat_last_cuda_error() -> int:
    return int(lib().hat_last_cuda_error())


def hat_launch_count() -> int:
    return int(lib().hat_launch_count())


def make_cache_desc(dtype, num_pages, num_kv_heads, head_dim, stride_page, stride_token, stride_head,
                    k_pool=None, v_pool=None, page_size=16) -> hat_cache_desc:
    code = DTYPE_CODE[dtype] if isinstance(dtype, str) else int(dtype)
    return hat_cache_desc(_ptr(k_pool), _ptr(v_pool), code, int(num_pages), int(page_size), int(num_kv_heads),
                          int(head_dim), 0, int(stride_page), int(stride_token), int(stride_head))


class Plan:
    """Owner of a hat_plan* (destroyed on close / garbage collection)."""

    def __init__(self, handle: int, keepalive):
        self.handle = handle
        self._keep = keepalive

    def close(self):
        if self.handle:
            hat_plan_destroy(self)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _h(plan) -> Optional[int]:
    return plan.handle if isinstance(plan, Plan) else plan


def hat_plan_create(cache: hat_cache_desc, num_q_heads: int, cu_chunk, prefix_len, chunk_len, block_table,
                    flags: int = 0, tree_mask=None) -> Plan:
    """The four arrays are host int32 arrays (numpy); block_table is [num_requests, max_pages]; tree_mask is
    None or a host uint32 array with one word per packed row."""
    cu = np.ascontiguousarray(cu_chunk, dtype=np.int32)
    pl = np.ascontiguousarray(prefix_len, dtype=np.int32)
    cl = np.ascontiguousarray(chunk_len, dtype=np.int32)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    R = int(pl.shape[0])
    max_pages = int(bt.shape[1]) if bt.ndim == 2 else 0
    tm = None if tree_mask is None else np.ascontiguousarray(tree_mask, dtype=np.uint32)
    batch = hat_batch_desc(R, int(num_q_heads), max_pages, int(flags), _ptr(cu), _ptr(pl), _ptr(cl),
                           _ptr(bt) if bt.size else None, None if tm is None or not tm.size else _ptr(tm))
    out = C.c_void_p()
    _check(lib().hat_plan_create(C.byref(cache), C.byref(batch), C.byref(out)), "hat_plan_create")
    return Plan(out.value, None)


def hat_plan_get_info(plan) -> hat_plan_info:
    info = hat_plan_info()
    _check(lib().hat_plan_get_info(_h(plan), C.byref(info)), "hat_plan_get_info")
    return info


def hat_plan_workspace_bytes(plan) -> int:
    n = C.c_size_t()
    _check(lib().hat_plan_workspace_bytes(_h(plan), C.byref(n)), "hat_plan_workspace_bytes")
    return int(n.value)


def hat_plan_staging_bytes(plan) -> int:
    n = C.c_size_t()
    _check(lib().hat_plan_staging_bytes(_h(plan), C.byref(n)), "hat_plan_staging_bytes")
    return int(n.value)


def hat_plan_destroy(plan) -> None:
    _check(lib().hat_plan_destroy(_h(plan)), "hat_plan_destroy")


def hat_kv_append(cache: hat_cache_desc, plan, k_new, v_new, stream: int = 0) -> None:
    _check(lib().hat_kv_append(C.byref(cache), _h(plan), _ptr(k_new), _ptr(v_new), stream or None), "hat_kv_append")


def hat_kv_append_rope(cache: hat_cache_desc, plan, k_new, v_new, theta: float = 10000.0, interleaved: bool = False,
                       stream: int = 0) -> None:
    _check(lib().hat_kv_append_rope(C.byref(cache), _h(plan), _ptr(k_new), _ptr(v_new), C.c_float(theta),
                                    int(bool(interleaved)), stream or None), "hat_kv_append_rope")


def hat_rope_q(plan, q, q_out, theta: float = 10000.0, interleaved: bool = False, stream: int = 0) -> None:
    _check(lib().hat_rope_q(_h(plan), _ptr(q), _ptr(q_out), C.c_float(theta), int(bool(interleaved)), stream or None),
           "hat_rope_q")


def hat_qkv_rope_append(cache: hat_cache_desc, plan, x, hidden: int, w_qkv, q_out, theta: float = 10000.0,
                        interleaved: bool = False, stream: int = 0) -> None:
    _check(lib().hat_qkv_rope_append(C.byref(cache), _h(plan), _ptr(x), int(hidden), _ptr(w_qkv), _ptr(q_out),
                                     C.c_float(theta), int(bool(interleaved)), stream or None), "hat_qkv_rope_append")


def hat_chunk_attention(cache: hat_cache_desc, plan, q, k_new, v_new, out, lse, sm_scale: float = 0.0,
                        workspace=None, workspace_bytes: int = 0, stream: int = 0) -> None:
    _check(lib().hat_chunk_attention(C.byref(cache), _h(plan), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                     _ptr(lse), float(sm_scale), _ptr(workspace), int(workspace_bytes),
                                     stream or None), "hat_chunk_attention")


def hat_chunk_attention_out16(cache: hat_cache_desc, plan, q, k_new, v_new, out16, lse, sm_scale: float = 0.0,
                              workspace=None, workspace_bytes: int = 0, stream: int = 0) -> None:
    _check(lib().hat_chunk_attention_out16(C.byref(cache), _h(plan), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out16),
                                           _ptr(lse), C.c_float(sm_scale), _ptr(workspace), workspace_bytes,
                                           stream or None), "hat_chunk_attention_out16")


def hat_chunk_attention_host(cache: hat_cache_desc, plan, q_host, k_new_host, v_new_host, out_host, lse_host,
                             sm_scale: float = 0.0, staging=None, staging_bytes: int = 0, workspace=None,
                             workspace_bytes: int = 0, stream: int = 0) -> None:
    _check(lib().hat_chunk_attention_host(C.byref(cache), _h(plan), _ptr(q_host), _ptr(k_new_host),
                                          _ptr(v_new_host), _ptr(out_host), _ptr(lse_host), float(sm_scale),
                                          _ptr(staging), int(staging_bytes), _ptr(workspace),
                                          int(workspace_bytes), stream or None), "hat_chunk_attention_host")


def hat_last_device_status(plan, stream: int = 0) -> int:
    st = C.c_int()
    _check(lib().hat_last_device_status(_h(plan), stream or None, C.byref(st)), "hat_last_device_status")
    return int(st.value)


def hat_plan_enable_timing(plan, max_calls: int) -> None:
    _check(lib().hat_plan_enable_timing(_h(plan), int(max_calls)), "hat_plan_enable_timing")


def hat_plan_read_timing(plan, capacity_calls: int) -> np.ndarray:
    """Per recorded call: milliseconds of [append, tile attention, streaming attention, merge]."""
    ms = np.zeros((int(capacity_calls), HAT_TIMING_SLOTS), dtype=np.float32)
    n = C.c_int()
    _check(lib().hat_plan_read_timing(_h(plan), _ptr(ms), int(capacity_calls), C.byref(n)), "hat_plan_read_timing")
    return ms[: n.value]


def hat_verify_attention_static(cache: hat_cache_desc, num_requests: int, num_q_heads: int, max_chunk_len: int,
                                max_pages: int, cu_chunk, prefix_len, chunk_len, block_table, q, out, lse,
                                sm_scale: float = 0.0, stream: int = 0) -> None:
    """Allocation-free streaming attention; the four descriptor arrays are DEVICE int32 tensors."""
    _check(lib().hat_verify_attention_static(C.byref(cache), int(num_requests), int(num_q_heads),
                                             int(max_chunk_len), int(max_pages), _ptr(cu_chunk), _ptr(prefix_len),
                                             _ptr(chunk_len), _ptr(block_table), _ptr(q), _ptr(out), _ptr(lse),
                                             float(sm_scale), stream or None), "hat_verify_attention_static")


def hat_static_key_range(prefix_len: int, chunk_len: int, max_chunk_len: int, max_pages: int, split: int):
    """(prefix, rows, kv_begin, kv_end) of one split of hat_verify_attention_static; host only."""
    o = [C.c_int32() for _ in range(4)]
    _check(lib().hat_static_key_range(int(prefix_len), int(chunk_len), int(max_chunk_len), int(max_pages), int(split),
                                      *[C.byref(x) for x in o]), "hat_static_key_range")
    return tuple(x.value for x in o)


def hat_plan_set_wait_limit(plan, cycles: int = 0, withhold_next_call: bool = False) -> None:
    _check(lib().hat_plan_set_wait_limit(_h(plan), int(cycles), 1 if withhold_next_call else 0),
           "hat_plan_set_wait_limit")


class Ctrl:
    """Owner of a hat_ctrl* (the cloud-side state monitor and chunk-size controller)."""

    def __init__(self, alpha: float = 0.8, bin_width: float = 64.0, num_bins: int = 256, max_devices: int = 64):
        h = C.c_void_p()
        _check(lib().hat_ctrl_create(alpha, bin_width, num_bins, max_devices, C.byref(h)), "hat_ctrl_create")
        self.handle = h.value

    def close(self):
        if self.handle:
            lib().hat_ctrl_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def hat_ctrl_observe(ctrl: Ctrl, mu_hat: float, eta_hat: float) -> None:
    _check(lib().hat_ctrl_observe(ctrl.handle, float(mu_hat), float(eta_hat)), "hat_ctrl_observe")


def hat_ctrl_mu(ctrl: Ctrl) -> float:
    v = C.c_double()
    _check(lib().hat_ctrl_mu(ctrl.handle, C.byref(v)), "hat_ctrl_mu")
    return v.value


def hat_ctrl_predict(ctrl: Ctrl, tokens: float) -> float:
    v = C.c_double()
    _check(lib().hat_ctrl_predict(ctrl.handle, float(tokens), C.byref(v)), "hat_ctrl_predict")
    return v.value


def hat_ctrl_device_observe(ctrl: Ctrl, device: int, gamma: float, beta_up: float, beta_down: float) -> None:
    _check(lib().hat_ctrl_device_observe(ctrl.handle, int(device), float(gamma), float(beta_up), float(beta_down)),
           "hat_ctrl_device_observe")


def hat_ctrl_device_state(ctrl: Ctrl, device: int):
    g, u, d = C.c_double(), C.c_double(), C.c_double()
    _check(lib().hat_ctrl_device_state(ctrl.handle, int(device), C.byref(g), C.byref(u), C.byref(d)),
           "hat_ctrl_device_state")
    return g.value, u.value, d.value


def hat_ctrl_chunk_size(ctrl: Ctrl, device: int, bytes_per_token: float, pipeline_length: int, x_min: int, x_max: int) -> int:
    v = C.c_int()
    _check(lib().hat_ctrl_chunk_size(ctrl.handle, int(device), float(bytes_per_token), int(pipeline_length), int(x_min),
                                     int(x_max), C.byref(v)), "hat_ctrl_chunk_size")
    return v.value


def hat_ctrl_parallel_draft_steps(ctrl: Ctrl, device: int, draft_len: int, bytes_per_token: float) -> int:
    v = C.c_int()
    _check(lib().hat_ctrl_parallel_draft_steps(ctrl.handle, int(device), int(draft_len), float(bytes_per_token),
                                               C.byref(v)), "hat_ctrl_parallel_draft_steps")
    return v.value


def hat_plan_verify_event(plan) -> int:
    """Raw cudaEvent_t recorded once the streaming-class rows of a call are final."""
    ev = C.c_void_p()
    _check(lib().hat_plan_verify_event(_h(plan), C.byref(ev)), "hat_plan_verify_event")
    return ev.value


def hat_plan_wait_verify(plan) -> None:
    _check(lib().hat_plan_wait_verify(_h(plan)), "hat_plan_wait_verify")
