"""Pins of the rotary-position oracle (CPU) and parity of the rotating append / query kernels (GPU)."""
import math
import types

import numpy as np
import pytest

from oracle import hat_oracle as O
from oracle import hat_rope_oracle as R
from paper_2503_18989_b200 import workloads as W

from common import assert_parity


# ----------------------------------------------------------------------------
# oracle pins
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("interleaved", [False, True])
def test_position_zero_is_the_identity_and_norms_are_kept(interleaved):
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 64))
    assert np.array_equal(R.rotate(x, np.zeros(5, np.int64), interleaved=interleaved), x)
    y = R.rotate(x, np.asarray([1, 17, 300, 4095, 8191]), interleaved=interleaved)
    assert np.allclose(np.sum(y * y, axis=-1), np.sum(x * x, axis=-1), rtol=1e-12)
    if interleaved:
        n_x, n_y = x[..., 0::2] ** 2 + x[..., 1::2] ** 2, y[..., 0::2] ** 2 + y[..., 1::2] ** 2
    else:
        n_x, n_y = x[..., :32] ** 2 + x[..., 32:] ** 2, y[..., :32] ** 2 + y[..., 32:] ** 2
    assert np.allclose(n_x, n_y, rtol=1e-12)          # every pair keeps its own norm


def test_hand_computed_pair():
    # d = 4, theta = 100: pair 0 turns by p radians, pair 1 by p / 10
    x = np.zeros((1, 1, 4)); x[0, 0] = [1.0, 2.0, 0.0, 1.0]        # half layout: pairs (x0, x2), (x1, x3)
    y = R.rotate(x, np.asarray([3]), theta=100.0)
    assert y[0, 0, 0] == pytest.approx(math.cos(3.0), abs=1e-15)
    assert y[0, 0, 2] == pytest.approx(math.sin(3.0), abs=1e-15)
    assert y[0, 0, 1] == pytest.approx(2 * math.cos(0.3) - math.sin(0.3), abs=1e-15)
    assert y[0, 0, 3] == pytest.approx(math.cos(0.3) + 2 * math.sin(0.3), abs=1e-15)
    z = R.rotate(x, np.asarray([3]), theta=100.0, interleaved=True)  # pairs (x0, x1), (x2, x3)
    assert z[0, 0, 0] == pytest.approx(math.cos(3.0) - 2 * math.sin(3.0), abs=1e-15)
    assert z[0, 0, 1] == pytest.approx(2 * math.cos(3.0) + math.sin(3.0), abs=1e-15)
    assert z[0, 0, 2] == pytest.approx(-math.sin(0.3), abs=1e-15)
    assert z[0, 0, 3] == pytest.approx(math.cos(0.3), abs=1e-15)


@pytest.mark.parametrize("interleaved", [False, True])
def test_rotations_compose_and_scores_depend_on_the_position_difference(interleaved):
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((4, 2, 128)), rng.standard_normal((4, 2, 128))
    a, b = np.asarray([5, 60, 700, 8000]), np.asarray([3, 11, 650, 1])
    twice = R.rotate(R.rotate(q, a, interleaved=interleaved), b, interleaved=interleaved)
    assert np.allclose(twice, R.rotate(q, a + b, interleaved=interleaved), atol=1e-10)
    s1 = np.sum(R.rotate(q, a, interleaved=interleaved) * R.rotate(k, b, interleaved=interleaved), axis=-1)
    s2 = np.sum(R.rotate(q, a - b + 1000, interleaved=interleaved) * R.rotate(k, np.full(4, 1000), interleaved=interleaved), axis=-1)
    assert np.allclose(s1, s2, atol=1e-9)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_rounding_to_the_storage_type(dtype):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = W.bits_to_f64(pats, dtype)
    ok = np.isfinite(vals)
    assert np.array_equal(R.round_to_bits(vals[ok], dtype), pats[ok])      # representable values map to themselves
    # halfway cases go to the even neighbour, everything else to the nearer one
    finite = pats[ok & (pats < 0x7B00)]                      # positive, below the top of both formats
    lo, hi = W.bits_to_f64(finite[:-1], dtype), W.bits_to_f64(finite[1:], dtype)
    mid = (lo + hi) / 2
    got = R.round_to_bits(mid, dtype)
    want = np.where(finite[:-1] % 2 == 0, finite[:-1], finite[1:])
    assert np.array_equal(got, want)
    assert np.array_equal(R.round_to_bits(lo + (hi - lo) * 0.49, dtype), finite[:-1])
    assert np.array_equal(R.round_to_bits(lo + (hi - lo) * 0.51, dtype), finite[1:])


def test_positions_follow_the_prefix():
    st = types.SimpleNamespace(num_requests=3, total_rows=7, prefix_len=np.asarray([10, 0, 5]),
                               cu_chunk=np.asarray([0, 3, 3, 7]))
    assert R.positions(st).tolist() == [10, 11, 12, 5, 6, 7, 8]


# ----------------------------------------------------------------------------
# GPU parity
# ----------------------------------------------------------------------------
def _assert_rotated(got_bits, want_bits, dtype, what, exact_share):
    """The fp32 rotation rounded once against the float64 rotation rounded once: equal bits nearly everywhere; where
    they differ, by one unit in the last place of the value, or, where the two products cancel, by the fp32 rounding of
    the products (inputs are below 8 in magnitude here: 8 * 2^-19 = 1.5e-5)."""
    got, want = W.bits_to_f64(got_bits, dtype), W.bits_to_f64(want_bits, dtype)
    assert np.isfinite(got).all(), what
    ulp = np.abs(want) * (2.0 ** -10 if dtype == "fp16" else 2.0 ** -7)          # at least one unit in the last place
    assert np.all(np.abs(got - want) <= ulp + 1.5e-5), (what, float(np.max(np.abs(got - want) - ulp)))
    share = float(np.mean(got_bits == want_bits))
    assert share > exact_share, (what, share)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,d,interleaved,group", [("fp16", 128, False, 1), ("bf16", 128, False, 4),
                                                       ("fp16", 64, True, 1), ("bf16", 64, True, 2)])
def test_rotating_append_and_query_kernels(cuda_device, dtype, d, interleaved, group):
    """hat_rope_q and hat_kv_append_rope against the float64 rotation rounded once: the same bits except where the
    fp32 result sits within rounding distance of a tie (at most one unit in the last place, rarely); then the whole
    step (rotated q, rotated cached K) against the oracle's attention over the oracle's own rotated cache."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    rng = np.random.Generator(np.random.PCG64(7))
    prefix, chunk = [0, 37, 1000, 4090, 8000, 250], [5, 16, 130, 40, 8, 0]
    table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=4)
    st = W._make_step(300, dtype, 2, d, prefix, chunk, table, q_heads=2 * group)
    sc = W._scenario("rope", dtype, 2, d, "paged", num_pages, [st], 300)
    pos = R.positions(st)
    theta = 10000.0

    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    q_rot = torch.empty_like(ds.q)
    B.hat_rope_q(ds.plan, ds.q, q_rot, theta, interleaved)
    B.hat_kv_append_rope(cache.desc, ds.plan, ds.k_new, ds.v_new, theta, interleaved)
    torch.cuda.synchronize()

    # (1) the rotated rows
    want_q = R.rope_bits(st.q, pos, dtype, theta, interleaved)
    got_q = q_rot.cpu().numpy().view(np.uint16).reshape(st.q.shape)
    _assert_rotated(got_q, want_q, dtype, "rotated q", 0.995)
    want_k = R.rope_bits(st.k_new, pos, dtype, theta, interleaved)
    ref = types.SimpleNamespace(**{**st.__dict__, "k_new": want_k})
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, ref)
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gv, vp), "V is stored as it comes"
    written = kp != sc.k_pool                                  # slots the oracle's append changed
    assert np.array_equal(gk[~written], kp[~written]), "a slot outside the chunk was written"
    _assert_rotated(gk[written], kp[written], dtype, "rotated K in the pool", 0.995)

    # (2) the step on top of it
    B.hat_chunk_attention(cache.desc, ds.plan, q_rot, None, None, ds.out, ds.lse, 0.0, ds.workspace,
                          ds.workspace_bytes)
    go, gl = ds.results()
    ref_step = types.SimpleNamespace(**{**st.__dict__, "q": want_q})
    wo, wl = O.chunk_attention(sc.cache, kp, vp, ref_step)
    assert_parity(go, wo, "rotated step out")
    assert_parity(gl, wl, "rotated step lse")
