"""ctypes front end of the CPU oracle (oracle/hat_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; never by the CUDA library or its binding.
All arithmetic lives in the C file; this module only marshals numpy arrays.
`cache` and `step` arguments are duck-typed (any object with the attributes
used below), so this module imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hat_oracle.c")
_LIB = os.path.join(_HERE, "libhat_oracle.so")
_lock = threading.Lock()
_lib = None

DTYPE_CODE = {"fp16": 0, "bf16": 1}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C + OpenMP); returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32, dbl, vp = C.c_int64, C.c_int, C.c_double, C.c_void_p
        L.hat_oracle_widen.restype = dbl
        L.hat_oracle_widen.argtypes = [C.c_uint16, i32]
        L.hat_oracle_kv_append.restype = None
        L.hat_oracle_kv_append.argtypes = [vp, vp, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp, i32, vp, vp]
        L.hat_oracle_attention_rows.restype = None
        L.hat_oracle_attention_rows.argtypes = [vp, vp, i32, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp, i32,
                                                vp, vp, dbl, i64, vp, vp, vp]
        L.hat_oracle_chunk_attention.restype = None
        L.hat_oracle_chunk_attention.argtypes = [vp, vp, i32, i64, i64, i64, i32, i32, i32, i32, i32, vp, vp, vp,
                                                 vp, i32, vp, vp, dbl, vp, vp]
        L.hat_oracle_merge.restype = None
        L.hat_oracle_merge.argtypes = [i32, i32, vp, vp, vp, vp]
        L.hat_oracle_threads.restype = i32
        L.hat_oracle_threads.argtypes = []
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def _c(a, dt) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dt)


def threads() -> int:
    return int(lib().hat_oracle_threads())


def widen(bits: int, dtype: str) -> float:
    return float(lib().hat_oracle_widen(int(bits), DTYPE_CODE[dtype]))


def kv_append(cache, k_pool: np.ndarray, v_pool: np.ndarray, step) -> None:
    """In-place append of step.k_new / step.v_new into the uint16 pools."""
    assert k_pool.dtype == np.uint16 and v_pool.dtype == np.uint16
    assert k_pool.flags.c_contiguous and v_pool.flags.c_contiguous
    cu, pl, cl = _c(step.cu_chunk, np.int32), _c(step.prefix_len, np.int32), _c(step.chunk_len, np.int32)
    bt = _c(step.block_table, np.int32)
    kn, vn = _c(step.k_new, np.uint16), _c(step.v_new, np.uint16)
    lib().hat_oracle_kv_append(_p(k_pool), _p(v_pool), cache.stride_page, cache.stride_token,
                               cache.stride_head, cache.page_size, cache.num_heads, cache.head_dim,
                               len(pl), _p(cu), _p(pl), _p(cl), _p(bt), bt.shape[1], _p(kn), _p(vn))


def _tree(step, T):
    """The step's optional tree mask as a contiguous uint32 [T] array (kept alive by the caller), or None."""
    tm = getattr(step, "tree_mask", None)
    if tm is None:
        return None
    tm = _c(tm, np.uint32)
    assert tm.shape == (T,)
    return tm


def chunk_attention(cache, k_pool, v_pool, step, sm_scale: float | None = None):
    """(out [T,Hq,d] float64, lse [T,Hq] float64) for every row of the batch; Hq = step.q.shape[1] query
    heads over cache.num_heads K/V heads."""
    Hkv, d = cache.num_heads, cache.head_dim
    H = int(step.q.shape[1])
    assert H % Hkv == 0
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(np.float64(d)))
    cu, pl, cl = _c(step.cu_chunk, np.int32), _c(step.prefix_len, np.int32), _c(step.chunk_len, np.int32)
    bt = _c(step.block_table, np.int32)
    q = _c(step.q, np.uint16)
    T = int(cu[-1])
    out = np.zeros((T, H, d), dtype=np.float64)
    lse = np.zeros((T, H), dtype=np.float64)
    tm = _tree(step, T)
    lib().hat_oracle_chunk_attention(_p(k_pool), _p(v_pool), DTYPE_CODE[cache.dtype], cache.stride_page,
                                     cache.stride_token, cache.stride_head, cache.page_size, Hkv, H, d,
                                     len(pl), _p(cu), _p(pl), _p(cl), _p(bt), bt.shape[1], _p(q),
                                     None if tm is None else _p(tm), float(sm_scale), _p(out), _p(lse))
    return out, lse


def attention_rows(cache, k_pool, v_pool, step, samples, sm_scale: float | None = None):
    """Attention for sampled rows.  `samples` is an array [n, 3] of (request, row, head) or
    [n, 5] of (request, row, query head, j_begin, j_end).  Returns (out [n, d], lse [n])."""
    Hkv, d = cache.num_heads, cache.head_dim
    H = int(step.q.shape[1])
    assert H % Hkv == 0
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(np.float64(d)))
    s = np.asarray(samples, dtype=np.int64)
    if s.ndim != 2 or s.shape[1] not in (3, 5):
        raise ValueError("samples must be [n,3] or [n,5]")
    if s.shape[1] == 3:
        s = np.concatenate([s, np.zeros((len(s), 1), np.int64), -np.ones((len(s), 1), np.int64)], axis=1)
    s = np.ascontiguousarray(s)
    cu, pl, cl = _c(step.cu_chunk, np.int32), _c(step.prefix_len, np.int32), _c(step.chunk_len, np.int32)
    bt = _c(step.block_table, np.int32)
    q = _c(step.q, np.uint16)
    out = np.zeros((len(s), d), dtype=np.float64)
    lse = np.zeros((len(s),), dtype=np.float64)
    tm = _tree(step, int(cu[-1]))
    lib().hat_oracle_attention_rows(_p(k_pool), _p(v_pool), DTYPE_CODE[cache.dtype], cache.stride_page,
                                    cache.stride_token, cache.stride_head, cache.page_size, Hkv, H, d,
                                    _p(cu), _p(pl), _p(cl), _p(bt), bt.shape[1], _p(q),
                                    None if tm is None else _p(tm), float(sm_scale),
                                    len(s), _p(s), _p(out), _p(lse))
    return out, lse


def merge(parts_out: np.ndarray, parts_lse: np.ndarray):
    """Merge partial results over disjoint key sets: parts_out [S, d], parts_lse [S]."""
    po, pl = _c(parts_out, np.float64), _c(parts_lse, np.float64)
    S, d = po.shape
    out = np.zeros(d, dtype=np.float64)
    lse = np.zeros(1, dtype=np.float64)
    lib().hat_oracle_merge(S, d, _p(po), _p(pl), _p(out), _p(lse))
    return out, float(lse[0])
