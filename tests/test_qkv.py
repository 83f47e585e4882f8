"""Pins of the projection oracle (CPU) and parity of the projection kernel with the rotation and the cache write in
its epilogue (GPU).  Paper Sec. 2.1: Q = X W_Q, K = X W_K, V = X W_V; K and V of every token stay in the KV cache."""
import types
from fractions import Fraction

import numpy as np
import pytest

from oracle import hat_oracle as O
from oracle import hat_qkv_oracle as QO
from oracle import hat_rope_oracle as R
from paper_2503_18989_b200 import workloads as W


def _bits(rng, shape, dtype, scale=1.0):
    return R.round_to_bits(rng.standard_normal(shape) * scale, dtype)


# ----------------------------------------------------------------------------
# oracle pins
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_projection_against_exact_rational_arithmetic(dtype):
    rng = np.random.default_rng(3)
    T, hidden, feats = 4, 9, 5                                 # not square, so a transposed operand cannot pass
    xb, wb = _bits(rng, (T, hidden), dtype), _bits(rng, (feats, hidden), dtype)
    y = QO.project(xb, wb, dtype)
    assert y.shape == (T, feats) and y.dtype == np.float64
    x, w = W.bits_to_f64(xb, dtype).reshape(T, hidden), W.bits_to_f64(wb, dtype).reshape(feats, hidden)
    for t in range(T):
        for f in range(feats):
            exact = sum(Fraction(float(x[t, j])) * Fraction(float(w[f, j])) for j in range(hidden))
            assert abs(Fraction(float(y[t, f])) - exact) <= abs(exact) * Fraction(1, 2 ** 50) + Fraction(1, 2 ** 60)


@pytest.mark.parametrize("dtype,d,interleaved,hq,hkv", [("fp16", 8, False, 3, 1), ("bf16", 4, True, 2, 2)])
def test_permutation_weights_reduce_to_the_pinned_rotation(dtype, d, interleaved, hq, hkv):
    """Weights with one entry 2^e per row: the projection is exact (y[t, f] = 2^e x[t, src[f]]), so the result has to
    be the rotation oracle applied to the gathered rows, bit for bit, and v the gathered rows themselves."""
    rng = np.random.default_rng(5)
    feats = (hq + 2 * hkv) * d
    hidden = feats + 3
    T = 6
    xb = _bits(rng, (T, hidden), dtype)
    src = rng.permutation(hidden)[:feats]
    e = rng.integers(-1, 2, size=feats)
    w = np.zeros((feats, hidden))
    w[np.arange(feats), src] = np.ldexp(1.0, e)
    wb = R.round_to_bits(w, dtype)
    pos = np.asarray([0, 1, 7, 130, 4099, 8000])
    qb, kb, vb = QO.qkv_rope(xb, wb, pos, dtype, hq, hkv, d, 10000.0, interleaved)
    x = W.bits_to_f64(xb, dtype).reshape(T, hidden)
    gathered = R.round_to_bits(x[:, src] * np.ldexp(1.0, e)[None, :], dtype)          # exact: a power of two
    gq = gathered[:, :hq * d].reshape(T, hq, d)
    gk = gathered[:, hq * d:(hq + hkv) * d].reshape(T, hkv, d)
    gv = gathered[:, (hq + hkv) * d:].reshape(T, hkv, d)
    assert np.array_equal(qb, R.rope_bits(gq, pos, dtype, 10000.0, interleaved))
    assert np.array_equal(kb, R.rope_bits(gk, pos, dtype, 10000.0, interleaved))
    assert np.array_equal(vb, gv)
    # without the rotation all three are the gathered rows
    q0, k0, v0 = QO.qkv_rope(xb, wb, pos, dtype, hq, hkv, d, None)
    assert np.array_equal(q0, gq) and np.array_equal(k0, gk) and np.array_equal(v0, gv)


def test_projection_is_additive_in_the_weights_and_rejects_bad_shapes():
    rng = np.random.default_rng(6)
    xb = _bits(rng, (5, 16), "fp16")
    w1, w2 = np.zeros((12, 16)), np.zeros((12, 16))
    w1[:, :8] = rng.integers(-4, 5, size=(12, 8))
    w2[:, 8:] = rng.integers(-4, 5, size=(12, 8))
    b1, b2, b12 = (R.round_to_bits(m, "fp16") for m in (w1, w2, w1 + w2))
    assert np.allclose(QO.project(xb, b12, "fp16"), QO.project(xb, b1, "fp16") + QO.project(xb, b2, "fp16"),
                       rtol=0, atol=1e-12)
    with pytest.raises(ValueError):
        QO.project(xb, b1[:, :15], "fp16")
    with pytest.raises(ValueError):
        QO.qkv_rope(xb, b1, np.zeros(5, np.int64), "fp16", 2, 1, 4)            # 12 rows are not (2 + 2) * 4
