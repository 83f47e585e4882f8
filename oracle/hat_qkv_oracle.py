"""CPU oracle for the step in front of the attention module: the Q/K/V projection of a decoder layer, the rotation of
the query and key rows by their position, and the write of the new key and value rows into the paged cache.

TEST INFRASTRUCTURE ONLY: shares no code with the CUDA library; only the tests load it.

Sec. 2.1 of the paper: an attention module multiplies the layer input X by three weight matrices, Q = X W_Q,
K = X W_K, V = X W_V, and the KV cache keeps K and V of every token seen so far.  The models of Sec. 4.1
(Vicuna-7B/13B) rotate Q and K by the token position before the scores are formed; that rotation is the one written
out in hat_rope_oracle.py and is reused here as a step.  Everything is float64 with ONE rounding to the 16-bit
storage type at the end:

    y[t, f]   = sum_j x[t, j] * w[f, j]                 w holds one row per output feature ([features][hidden]), i.e.
                                                        the transpose of the paper's W_Q | W_K | W_V side by side
    features  = [ Hq heads of q | Hkv heads of k | Hkv heads of v ], d values each
    q, k      rotated by the row's position (hat_rope_oracle.rotate), v as it comes
    k, v      go to slot (prefix_len[r] + i) of request r's pages (the append of hat_oracle)

Pins (tests/test_qkv.py): the sum against exact rational arithmetic on small shapes; weights that are a permutation
(times powers of two) of the inputs, where the projection is exact and the result must equal the pinned rotation of
the permuted rows bit for bit (a transposed operand or a wrong head offset fails it); additivity in the weights.
"""
from __future__ import annotations

import numpy as np

from . import hat_rope_oracle as R


def project(x_bits: np.ndarray, w_bits: np.ndarray, dtype: str) -> np.ndarray:
    """x: [T, hidden] bit patterns, w: [features, hidden] bit patterns.  Returns y = x w^T in float64, [T, features]."""
    x = R.bits_to_f64(x_bits, dtype).reshape(x_bits.shape)
    w = R.bits_to_f64(w_bits, dtype).reshape(w_bits.shape)
    if x.shape[1] != w.shape[1]:
        raise ValueError("x and w disagree on the hidden size")
    return x @ w.T


def qkv_rope(x_bits: np.ndarray, w_bits: np.ndarray, pos: np.ndarray, dtype: str, q_heads: int, kv_heads: int,
             head_dim: int, theta: float | None = 10000.0, interleaved: bool = False):
    """The projected rows split into heads, q and k rotated (theta None: no rotation), rounded once.

    Returns (q_bits [T, q_heads, d], k_bits [T, kv_heads, d], v_bits [T, kv_heads, d]) as uint16 bit patterns."""
    T = x_bits.shape[0]
    d = head_dim
    if w_bits.shape[0] != (q_heads + 2 * kv_heads) * d:
        raise ValueError("w has the wrong number of rows")
    y = project(x_bits, w_bits, dtype)
    q = y[:, :q_heads * d].reshape(T, q_heads, d)
    k = y[:, q_heads * d:(q_heads + kv_heads) * d].reshape(T, kv_heads, d)
    v = y[:, (q_heads + kv_heads) * d:].reshape(T, kv_heads, d)
    if theta is not None:
        q = R.rotate(q, pos, theta, interleaved)
        k = R.rotate(k, pos, theta, interleaved)
    return R.round_to_bits(q, dtype), R.round_to_bits(k, dtype), R.round_to_bits(v, dtype)
