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


# ----------------------------------------------------------------------------
# GPU parity
# ----------------------------------------------------------------------------
def _assert_projected(got_bits, want_bits, dtype, what, exact_share):
    """fp32 accumulation on the tensor cores, fp32 rotation, one rounding, against float64 rounded once: the same bits
    nearly everywhere; elsewhere within one unit in the last place plus the accumulation error (hidden <= 5120 terms
    of magnitude <= 1, each step rounded to 2^-23 of a partial sum of a few units: below 2e-4)."""
    got, want = W.bits_to_f64(got_bits, dtype), W.bits_to_f64(want_bits, dtype)
    assert np.isfinite(got).all(), what
    ulp = np.abs(want) * (2.0 ** -10 if dtype == "fp16" else 2.0 ** -7)
    worst = float(np.max(np.abs(got - want) - ulp))
    assert worst <= 2e-4, (what, worst)
    share = float(np.mean(got_bits == want_bits))
    assert share > exact_share, (what, share)


def _run_projection(cuda_device, dtype, d, hq, hkv, hidden, prefix, chunk, theta, interleaved, seed=11):
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    rng = np.random.Generator(np.random.PCG64(seed))
    table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=4)
    st = W._make_step(500 + seed, dtype, hkv, d, prefix, chunk, table, q_heads=hq)
    sc = W._scenario("qkv", dtype, hkv, d, "paged", num_pages, [st], 500 + seed)
    T = st.total_rows
    feats = (hq + 2 * hkv) * d
    xb, wb = W.projection_inputs(700 + seed, dtype, T, hidden, feats)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x_dev = runner._dev_u16(xb, cuda_device)
    w_dev = runner._dev_u16(wb, cuda_device)
    g_q = runner._Guarded((T, hq, d), torch.int16, -1, cuda_device)
    B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, g_q.view, theta, interleaved)
    torch.cuda.synchronize()
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    assert g_q.intact(), "a canary zone around q_out was overwritten"
    got_q = g_q.view.cpu().numpy().view(np.uint16).reshape(T, hq, d)
    gk, gv = cache.pools_to_host()
    return sc, st, ds, cache, xb, wb, got_q, gk, gv


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,d,hq,hkv,hidden,theta,interleaved,small", [
    ("fp16", 128, 4, 2, 448, 10000.0, False, False),   # 4 feature tiles, 7 stages of the hidden dimension (the ring wraps)
    ("bf16", 128, 2, 2, 64, 10000.0, True, False),     # one stage per tile
    ("bf16", 64, 6, 3, 128, 10000.0, True, False),     # four heads per feature tile
    ("fp16", 64, 3, 1, 192, 500000.0, False, False),   # 320 features: the second feature tile is partly empty
    ("fp16", 128, 3, 1, 128, 0.0, False, False),       # no rotation; 5 heads: the last tile holds one
    ("bf16", 128, 4, 2, 320, 10000.0, False, True),    # at most 128 rows: the one-CTA form (5 stages, ring of 4)
    ("fp16", 64, 3, 1, 64, 10000.0, True, True),
])
def test_projection_kernel_rotates_and_appends(cuda_device, dtype, d, hq, hkv, hidden, theta, interleaved, small):
    """hat_qkv_rope_append against the float64 projection, rotation and append: q rows, the written slots of both
    pools (and nothing but them).  359 rows (CTA pairs, a ragged second pair of row tiles) or 100 rows (single CTAs)."""
    prefix, chunk = ([0, 37, 4090], [5, 80, 15]) if small else ([0, 37, 1000, 4090, 8000, 250], [5, 130, 16, 200, 8, 0])
    sc, st, ds, cache, xb, wb, got_q, gk, gv = _run_projection(cuda_device, dtype, d, hq, hkv, hidden, prefix, chunk,
                                                               theta, interleaved)
    pos = R.positions(st)
    want_q, want_k, want_v = QO.qkv_rope(xb, wb, pos, dtype, hq, hkv, d, theta if theta > 0 else None, interleaved)
    _assert_projected(got_q, want_q, dtype, "q rows", 0.97)
    ref = types.SimpleNamespace(**{**st.__dict__, "k_new": want_k, "v_new": want_v})
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, ref)
    # slots of the chunk rows: found by appending a marker pattern through the oracle
    mark = types.SimpleNamespace(**{**st.__dict__, "k_new": np.full_like(want_k, 0xFFFF), "v_new": np.full_like(want_v, 0xFFFF)})
    mk, mv = np.zeros_like(kp), np.zeros_like(vp)
    O.kv_append(sc.cache, mk, mv, mark)
    written = mk == 0xFFFF
    assert written.sum() == want_k.size
    assert np.array_equal(gk[~written], sc.k_pool[~written]), "a K slot outside the chunk was written"
    assert np.array_equal(gv[~written], sc.v_pool[~written]), "a V slot outside the chunk was written"
    _assert_projected(gk[written], kp[written], dtype, "K in the pool", 0.97)
    _assert_projected(gv[written], vp[written], dtype, "V in the pool", 0.97)
    ds.close()


@pytest.mark.gpu
def test_projection_then_attention_matches_the_oracle_step(cuda_device):
    """The whole layer front: projection kernel, then hat_chunk_attention on its q rows and the cache it wrote, against
    the oracle's attention over the oracle's own projected, rotated and appended rows."""
    import torch
    from paper_2503_18989_b200 import binding as B
    from common import assert_parity
    dtype, d, hq, hkv, hidden = "bf16", 128, 4, 2, 256
    prefix, chunk = [0, 300, 2000], [256, 4, 70]
    sc, st, ds, cache, xb, wb, got_q, gk, gv = _run_projection(cuda_device, dtype, d, hq, hkv, hidden, prefix, chunk,
                                                               10000.0, False, seed=12)
    q_dev = torch.from_numpy(got_q.view(np.int16)).to(cuda_device)
    B.hat_chunk_attention(cache.desc, ds.plan, q_dev, None, None, ds.out, ds.lse, 0.0, ds.workspace, ds.workspace_bytes)
    go, gl = ds.results()
    want_q, want_k, want_v = QO.qkv_rope(xb, wb, R.positions(st), dtype, hq, hkv, d)
    ref = types.SimpleNamespace(**{**st.__dict__, "q": want_q, "k_new": want_k, "v_new": want_v})
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, ref)
    wo, wl = O.chunk_attention(sc.cache, kp, vp, ref)
    assert_parity(go, wo, "layer front out")
    assert_parity(gl, wl, "layer front lse")
    ds.close()


@pytest.mark.gpu
def test_projection_kernel_rejects_what_it_cannot_run(cuda_device):
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    rng = np.random.Generator(np.random.PCG64(3))
    table, num_pages = W._place_pages(rng, np.asarray([20]), slack_pages=1)
    st = W._make_step(1, "fp16", 1, 128, [4], [16], table, q_heads=1)
    sc = W._scenario("qkv", "fp16", 1, 128, "paged", num_pages, [st], 1)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x = torch.zeros(16 * 96, dtype=torch.int16, device=cuda_device)
    w = torch.zeros(384 * 96, dtype=torch.int16, device=cuda_device)
    q = torch.zeros(16 * 128, dtype=torch.int16, device=cuda_device)
    L = B.lib()
    import ctypes as C
    def call(hidden, theta, xp=x):
        return L.hat_qkv_rope_append(C.byref(cache.desc), B._h(ds.plan), B._ptr(xp), hidden, B._ptr(w), B._ptr(q),
                                     C.c_float(theta), 0, None)
    assert call(96, 10000.0) == B.HAT_ERR_UNSUPPORTED                            # hidden not a multiple of 64
    assert call(64, 0.5) == B.HAT_ERR_INVALID_ARG                                # a base in (0, 1]
    assert call(0, 10000.0) == B.HAT_ERR_INVALID_ARG
    assert call(64, 10000.0, xp=None) == B.HAT_ERR_INVALID_ARG
    assert call(64, 10000.0) == B.HAT_OK
    torch.cuda.synchronize()
    ds.close()


@pytest.mark.gpu
def test_projection_at_the_13b_mixed_batch_size_on_sampled_rows(cuda_device):
    """The projection of the 13B-shaped mixed batch (4224 rows, hidden 5120, 40 + 40 + 40 heads of 128, bf16) in the
    launch configuration the benchmark times: sampled rows (first and last row of prefill and verify requests, random
    others) against the float64 oracle, q rows and the K / V slots read back through the block table."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    sc = W.mixed_13b()
    st = sc.steps[0]
    spec = sc.cache
    dtype, d, hkv = spec.dtype, spec.head_dim, spec.num_heads
    hq = int(st.q.shape[1])
    hidden = hq * d
    T = st.total_rows
    feats = (hq + 2 * hkv) * d
    xb, wb = W.projection_inputs(900, dtype, T, hidden, feats)
    cache = runner.DeviceCache(spec, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x_dev, w_dev = runner._dev_u16(xb, cuda_device), runner._dev_u16(wb, cuda_device)
    g_q = runner._Guarded((T, hq, d), torch.int16, -1, cuda_device)
    B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, g_q.view, 10000.0, False)
    torch.cuda.synchronize()
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    assert g_q.intact()

    rng = np.random.default_rng(4)
    pos = R.positions(st)
    rows = set(int(t) for t in rng.integers(0, T, size=24))
    for r in list(range(0, st.num_requests, 7)) + [st.num_requests - 1]:
        if st.chunk_len[r] > 0:
            rows.update((int(st.cu_chunk[r]), int(st.cu_chunk[r + 1]) - 1))
    rows = np.asarray(sorted(rows))
    req = np.searchsorted(st.cu_chunk, rows, side="right") - 1
    want_q, want_k, want_v = QO.qkv_rope(xb[rows], wb, pos[rows], dtype, hq, hkv, d)
    got_q = g_q.view[torch.from_numpy(rows).to(cuda_device)].cpu().numpy().view(np.uint16)
    _assert_projected(got_q, want_q, dtype, "sampled q rows", 0.97)
    # element offsets of the sampled rows' slots: [row][head][d]
    page = st.block_table[req, pos[rows] // spec.page_size].astype(np.int64)
    base = page * spec.stride_page + (pos[rows] % spec.page_size) * spec.stride_token
    offs = base[:, None, None] + (np.arange(hkv, dtype=np.int64) * spec.stride_head)[None, :, None] + np.arange(d)[None, None, :]
    idx = torch.from_numpy(offs.reshape(-1)).to(cuda_device)
    got_k = cache.k.view(-1)[idx].cpu().numpy().view(np.uint16).reshape(len(rows), hkv, d)
    got_v = cache.v.view(-1)[idx].cpu().numpy().view(np.uint16).reshape(len(rows), hkv, d)
    _assert_projected(got_k, want_k, dtype, "sampled K slots", 0.97)
    _assert_projected(got_v, want_v, dtype, "sampled V slots", 0.97)
    # the slot behind a request's last row belongs to nobody yet and keeps its content
    for r in (0, st.num_requests - 1):
        p_next = int(st.prefix_len[r] + st.chunk_len[r])
        if p_next // spec.page_size < st.max_pages and st.block_table[r, p_next // spec.page_size] >= 0:
            o = int(st.block_table[r, p_next // spec.page_size]) * spec.stride_page + (p_next % spec.page_size) * spec.stride_token
            assert np.array_equal(cache.k.view(-1)[o:o + d].cpu().numpy().view(np.uint16), sc.k_pool[o:o + d])
    ds.close()


@pytest.mark.gpu
def test_projection_on_two_streams_and_with_two_bases(cuda_device):
    """The table of cosines and sines belongs to the plan: a call on another stream than the one that filled it is
    ordered behind the fill, and a call with another base refills it.  Same results as single-stream calls."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    dtype, d, hq, hkv, hidden = "fp16", 128, 2, 1, 128
    prefix, chunk = [0, 500, 4000], [140, 3, 60]
    rng = np.random.Generator(np.random.PCG64(21))
    table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=2)
    st = W._make_step(321, dtype, hkv, d, prefix, chunk, table, q_heads=hq)
    sc = W._scenario("qkv", dtype, hkv, d, "paged", num_pages, [st], 321)
    T = st.total_rows
    xb, wb = W.projection_inputs(55, dtype, T, hidden, (hq + 2 * hkv) * d)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x_dev, w_dev = runner._dev_u16(xb, cuda_device), runner._dev_u16(wb, cuda_device)
    s1, s2 = torch.cuda.Stream(cuda_device), torch.cuda.Stream(cuda_device)
    torch.cuda.synchronize()
    pos = R.positions(st)
    outs = {}
    for theta, stream in ((10000.0, s1), (10000.0, s2), (500000.0, s2), (500000.0, s1)):
        q = torch.full((T, hq, d), -1, dtype=torch.int16, device=cuda_device)
        B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q, theta, False, stream.cuda_stream)
        outs.setdefault(theta, []).append(q)
    torch.cuda.synchronize()
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    for theta, qs in outs.items():
        want_q, _, _ = QO.qkv_rope(xb, wb, pos, dtype, hq, hkv, d, theta)
        a, b = (t.cpu().numpy().view(np.uint16) for t in qs)
        assert np.array_equal(a, b), "the same call on another stream gives other bits"
        _assert_projected(a, want_q, dtype, f"q rows, base {theta}", 0.97)
    ds.close()


@pytest.mark.gpu
@pytest.mark.parametrize("rows", [300, 100])
def test_projection_kernel_gives_up_a_wait_and_the_context_stays_usable(cuda_device, rows):
    """Failure detection without a fault: the producer of CTA 0 (of every pair; 300 rows run on pairs, 100 on single
    CTAs) withholds its first transfer, the waits on it run out after the shortened bound, both CTAs of a pair wind
    down, the status word reports it, reading clears it, and the next call is correct."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    dtype, d, hq, hkv, hidden = "fp16", 128, 2, 1, 512
    prefix, chunk = [40, 900], [rows - 20, 20]
    rng = np.random.Generator(np.random.PCG64(31))
    table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=2)
    st = W._make_step(77, dtype, hkv, d, prefix, chunk, table, q_heads=hq)
    sc = W._scenario("qkv", dtype, hkv, d, "paged", num_pages, [st], 77)
    T = st.total_rows
    xb, wb = W.projection_inputs(66, dtype, T, hidden, (hq + 2 * hkv) * d)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x_dev, w_dev = runner._dev_u16(xb, cuda_device), runner._dev_u16(wb, cuda_device)
    q = torch.full((T, hq, d), -1, dtype=torch.int16, device=cuda_device)
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    B.hat_plan_set_wait_limit(ds.plan, 20_000_000, withhold_next_call=True)      # about 10 ms
    B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q, 10000.0, False)
    assert B.hat_last_device_status(ds.plan) == B.HAT_ERR_DEVICE_TIMEOUT
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK                          # reading cleared it
    B.hat_plan_set_wait_limit(ds.plan, 0, withhold_next_call=False)
    B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q, 10000.0, False)
    torch.cuda.synchronize()
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    want_q, _, _ = QO.qkv_rope(xb, wb, R.positions(st), dtype, hq, hkv, d)
    _assert_projected(q.cpu().numpy().view(np.uint16), want_q, dtype, "q rows after the self test", 0.97)
    ds.close()


@pytest.mark.gpu
def test_projection_call_captured_in_a_cuda_graph(cuda_device):
    """The call neither allocates nor synchronises, so it can be captured; the captured graph carries its own fill of
    the cosine / sine table, and a direct call afterwards (which finds the plan's table not yet filled) is correct too."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    dtype, d, hq, hkv, hidden = "bf16", 128, 2, 2, 192
    prefix, chunk = [10, 777], [150, 40]
    rng = np.random.Generator(np.random.PCG64(41))
    table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=2)
    st = W._make_step(91, dtype, hkv, d, prefix, chunk, table, q_heads=hq)
    sc = W._scenario("qkv", dtype, hkv, d, "paged", num_pages, [st], 91)
    T = st.total_rows
    xb, wb = W.projection_inputs(92, dtype, T, hidden, (hq + 2 * hkv) * d)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    x_dev, w_dev = runner._dev_u16(xb, cuda_device), runner._dev_u16(wb, cuda_device)
    q = torch.full((T, hq, d), -1, dtype=torch.int16, device=cuda_device)
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(torch.cuda.current_stream(cuda_device))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q, 10000.0, False, side.cuda_stream)
    want_q, _, _ = QO.qkv_rope(xb, wb, R.positions(st), dtype, hq, hkv, d)
    for _ in range(2):
        q.fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        _assert_projected(q.cpu().numpy().view(np.uint16), want_q, dtype, "q rows from the replayed graph", 0.97)
    q.fill_(-1)
    B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q, 10000.0, False)      # direct call after the capture
    torch.cuda.synchronize()
    _assert_projected(q.cpu().numpy().view(np.uint16), want_q, dtype, "q rows from a direct call", 0.97)
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    ds.close()
