"""CPU oracle for rotary position encoding of the rows that enter the KV cache and of the query rows.

TEST INFRASTRUCTURE ONLY: shares no code with the CUDA library; only the tests load it.

The paper does not spell out the position encoding: its models are Vicuna-7B/13B (Sec. 4.1), whose decoder layers
rotate the query and key rows by their token position before the attention module of Sec. 2.1, and the key rows are
cached after that rotation (Sec. 2.1, KV cache).  This file is that rotation written out in float64, followed by ONE
rounding to the 16-bit storage type:

    position of chunk row i of request r:   p = prefix_len[r] + i
    angle of pair c (c = 0 .. d/2 - 1):     a = p * theta ** (-2 c / d)
    the pair (x_lo, x_hi) becomes           (x_lo cos a - x_hi sin a,  x_hi cos a + x_lo sin a)
    pairs:  "half"        x_lo = x[c],   x_hi = x[c + d/2]      (the layout of the Vicuna / LLaMA checkpoints)
            "interleaved" x_lo = x[2c],  x_hi = x[2c + 1]

Pins (tests/test_rope.py): position 0 is the identity; norms of pairs are preserved; composition of two rotations;
the score of a rotated query with a rotated key depends on the position difference only; a hand-computed pair.
"""
from __future__ import annotations

import numpy as np


def bits_to_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    """fp16 / bf16 bit patterns widened exactly to float64 (the oracle's own decoder)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "fp16":
        return bits.view(np.float16).astype(np.float64)
    if dtype != "bf16":
        raise ValueError(dtype)
    # a bf16 pattern is the upper half of the float32 with the same value
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def round_to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """float64 -> fp16 / bf16 bit patterns, round to nearest even, straight from float64 (no float32 step)."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "fp16":
        return x.astype(np.float16).view(np.uint16)
    if dtype != "bf16":
        raise ValueError(dtype)
    # bf16: 8 significant bits, exponent range of float32.  Quantum of a value with binary exponent e is 2^(e-7).
    out = np.where(x == 0, x, 0.0)                 # zeros keep their sign
    nz = (x != 0) & np.isfinite(x)
    m, e = np.frexp(x[nz])                         # x = m * 2^e, 0.5 <= |m| < 1  =>  binary exponent e - 1
    e = np.maximum(e - 1, -126)                    # subnormals share the smallest normal exponent
    q = np.ldexp(1.0, e - 7)
    out[nz] = np.rint(x[nz] / q) * q               # rint rounds half to even
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    f32 = out.astype(np.float32)                   # exact: the value has at most 8 significant bits
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def positions(step) -> np.ndarray:
    """Token position of every packed row of the step."""
    pos = np.zeros(step.total_rows, dtype=np.int64)
    for r in range(step.num_requests):
        a, b = int(step.cu_chunk[r]), int(step.cu_chunk[r + 1])
        pos[a:b] = int(step.prefix_len[r]) + np.arange(b - a)
    return pos


def rotate(x: np.ndarray, pos: np.ndarray, theta: float = 10000.0, interleaved: bool = False) -> np.ndarray:
    """x: float64 [T, H, d]; pos: [T].  Returns the rotated rows, float64."""
    T, H, d = x.shape
    half = d // 2
    c = np.arange(half, dtype=np.float64)
    ang = pos.astype(np.float64)[:, None] * np.power(np.float64(theta), -2.0 * c / d)[None, :]    # [T, d/2]
    cs, sn = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    out = np.empty_like(x)
    if interleaved:
        lo, hi = x[..., 0::2], x[..., 1::2]
        out[..., 0::2] = lo * cs - hi * sn
        out[..., 1::2] = hi * cs + lo * sn
    else:
        lo, hi = x[..., :half], x[..., half:]
        out[..., :half] = lo * cs - hi * sn
        out[..., half:] = hi * cs + lo * sn
    return out


def rope_bits(bits: np.ndarray, pos: np.ndarray, dtype: str, theta: float = 10000.0,
              interleaved: bool = False) -> np.ndarray:
    """16-bit rows in, rotated 16-bit rows out (one rounding)."""
    x = bits_to_f64(bits, dtype).reshape(bits.shape)
    return round_to_bits(rotate(x, pos, theta, interleaved), dtype)
