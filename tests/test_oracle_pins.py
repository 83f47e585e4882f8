"""Pins for the CPU oracle: closed forms, invariants, brute force and a library cross-check.

None of these compares the oracle with itself through the same code path: each
pins it to a value fixed by the mathematics (closed form), to an independent
evaluation (pure-Python brute force, a library SDPA routine on a dense special
case), or to an invariant a wrong index / mask / sign would break.
"""
import math
import types

import numpy as np
import pytest

from oracle import hat_oracle as O
from paper_2503_18989_b200 import workloads as W


def _cache(dtype, H, d, num_pages, layout):
    return W.CacheSpec(dtype, H, d, num_pages, layout)


def _step(prefix, chunk, table, q, k, v):
    prefix = np.asarray(prefix, np.int32)
    chunk = np.asarray(chunk, np.int32)
    cu = np.zeros(len(chunk) + 1, np.int32)
    cu[1:] = np.cumsum(chunk)
    return types.SimpleNamespace(prefix_len=prefix, chunk_len=chunk, cu_chunk=cu,
                                 block_table=np.asarray(table, np.int32), q=q, k_new=k, v_new=v)


def _bits(x, dtype="fp16"):
    return W.f32_to_bits(np.asarray(x, np.float32), dtype)


# ----------------------------------------------------------------------------
# 16-bit decoding
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_widen_all_patterns(dtype):
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = W.bits_to_f64(pats, dtype)     # numpy's own decoders
    got = np.array([O.widen(int(p), dtype) for p in pats])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


# ----------------------------------------------------------------------------
# closed forms
# ----------------------------------------------------------------------------
def test_two_key_closed_form():
    # d=64 so sm_scale = 1/8.  q=(8,0,..), k0=0, k1=(1,0,..) => scores (0, 1).
    # Weights 1/(1+e), e/(1+e); v0=e_0, v1=e_1 => out=(1/(1+e), e/(1+e), 0..), lse=ln(1+e).
    H, d = 1, 64
    cache = _cache("fp16", H, d, 1, "contiguous")
    k = np.zeros((16, H, d), np.float32); v = np.zeros((16, H, d), np.float32)
    k[1, 0, 0] = 1.0; v[0, 0, 0] = 1.0; v[1, 0, 1] = 1.0
    k[2, 0, 0] = 30.0; v[2, 0, 2] = 5.0        # position 2 is NOT visible to row 0 at prefix 1
    q = np.zeros((1, H, d), np.float32); q[0, 0, 0] = 8.0
    st = _step([1], [1], [[0]], _bits(q), _bits(k[1:2]), _bits(v[1:2]))
    out, lse = O.chunk_attention(cache, _bits(k).ravel(), _bits(v).ravel(), st)
    e = math.e
    assert out[0, 0, 0] == pytest.approx(1 / (1 + e), abs=1e-15)
    assert out[0, 0, 1] == pytest.approx(e / (1 + e), abs=1e-15)
    assert np.all(out[0, 0, 2:] == 0.0)
    assert lse[0, 0] == pytest.approx(math.log(1 + e), abs=1e-15)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_zero_query_gives_mean_of_visible_values(dtype):
    # Q = 0 => all scores 0 => out = mean(V[0..P+i]), lse = ln(P+i+1).
    sc = W.tiny(prompt=96, chunk=32, draft=5, H=3, d=64, dtype=dtype, seed=7)
    cache = sc.cache
    V = W.bits_to_f64(sc.v_pool, dtype).reshape(-1, cache.num_heads, cache.head_dim)  # contiguous layout
    for st in sc.steps:
        st.q[:] = 0
        P, Cn = int(st.prefix_len[0]), int(st.chunk_len[0])
        out, lse = O.chunk_attention(cache, sc.k_pool, sc.v_pool, st)
        for i in range(Cn):
            n = P + i + 1
            want = V[:n].sum(axis=0) / n
            assert np.allclose(out[i], want, rtol=0, atol=1e-13)
            assert np.allclose(lse[i], math.log(n), rtol=0, atol=1e-13)


def test_first_row_sees_only_itself():
    sc = W.tiny(prompt=16, chunk=16, draft=1, H=2, d=64, seed=11)
    cache, st = sc.cache, sc.steps[0]
    out, lse = O.chunk_attention(cache, sc.k_pool, sc.v_pool, st)
    V = W.bits_to_f64(sc.v_pool, "fp16").reshape(-1, 2, 64)
    K = W.bits_to_f64(sc.k_pool, "fp16").reshape(-1, 2, 64)
    Q = W.bits_to_f64(st.q, "fp16")
    assert np.array_equal(out[0], V[0])
    s0 = (Q[0] * K[0]).sum(-1) / 8.0
    assert np.allclose(lse[0], s0, rtol=0, atol=1e-13)


def test_constant_values_and_dominant_key():
    H, d, n = 2, 64, 40
    cache = _cache("fp16", H, d, 3, "contiguous")
    rng = np.random.default_rng(5)
    k = rng.standard_normal((48, H, d)).astype(np.float32)
    q = rng.standard_normal((1, H, d)).astype(np.float32)
    v = np.full((48, H, d), 0.375, np.float32)
    st = _step([n - 1], [1], [[0, 1, 2]], _bits(q), _bits(k[n - 1:n]), _bits(v[n - 1:n]))
    out, _ = O.chunk_attention(cache, _bits(k).ravel(), _bits(v).ravel(), st)
    assert np.allclose(out, 0.375, rtol=0, atol=1e-15)
    # one key aligned with q and scaled up takes all the weight
    v = rng.standard_normal((48, H, d)).astype(np.float32)
    k[17] = 40.0 * q[0] / np.linalg.norm(q[0], axis=-1, keepdims=True)
    qq = 40.0 * q / np.linalg.norm(q[0], axis=-1, keepdims=True)
    out, _ = O.chunk_attention(cache, _bits(k).ravel(), _bits(v).ravel(),
                               _step([n - 1], [1], [[0, 1, 2]], _bits(qq), _bits(k[n - 1:n]), _bits(v[n - 1:n])))
    want = W.bits_to_f64(_bits(v[17]), "fp16")
    assert np.allclose(out[0], want, rtol=0, atol=1e-9)


# ----------------------------------------------------------------------------
# brute force in pure Python (independent indexing, three passes, fsum)
# ----------------------------------------------------------------------------
def _brute_row(cache, k_pool, v_pool, st, r, i, h):
    """h is the query head; with grouped query heads it reads K/V head h // G.  A tree mask, if the step has
    one and the chunk is short, picks the visible chunk positions."""
    d = cache.head_dim
    kf = W.bits_to_f64(k_pool, cache.dtype); vf = W.bits_to_f64(v_pool, cache.dtype)
    qf = W.bits_to_f64(st.q, cache.dtype)
    row = int(st.cu_chunk[r]) + i
    hk = h // (st.q.shape[1] // cache.num_heads)
    P, Cn = int(st.prefix_len[r]), int(st.chunk_len[r])
    tm = getattr(st, "tree_mask", None)
    if tm is not None and Cn <= 16:
        visible = list(range(P)) + [P + c for c in range(Cn) if (int(tm[row]) >> c) & 1]
    else:
        visible = list(range(P + i + 1))
    scores = []
    addr = []
    for j in visible:
        page = int(st.block_table[r][j // cache.page_size])
        a = page * cache.stride_page + (j % cache.page_size) * cache.stride_token + hk * cache.stride_head
        addr.append(a)
        scores.append(math.fsum(float(qf[row, h, c]) * float(kf[a + c]) for c in range(d)) / math.sqrt(d))
    top = max(scores)
    wts = [math.exp(s - top) for s in scores]
    tot = math.fsum(wts)
    out = [math.fsum(w * float(vf[a + c]) for w, a in zip(wts, addr)) / tot for c in range(d)]
    return np.array(out), top + math.log(tot)


@pytest.mark.parametrize("maker,kw", [
    (W.ragged_prefill, dict(num_requests=3, max_prefix=48, chunk_choices=(5, 16, 23), H=2, d=64, seed=3)),
    (W.spec_verify, dict(num_requests=3, min_prefix=3, max_prefix=70, max_draft=8, H=2, d=64, seed=4)),
    (W.mixed_13b, dict(num_prefill=1, prefill_chunk=20, max_prefill_prefix=40, num_verify=2, draft=4,
                       min_verify_prefix=10, max_verify_prefix=50, H=2, d=128, seed=6)),
])
def test_brute_force_rows(maker, kw):
    sc = maker(**kw)
    cache, st = sc.cache, sc.steps[0]
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(cache, kp, vp, st)
    out, lse = O.chunk_attention(cache, kp, vp, st)
    rng = np.random.default_rng(1)
    for _ in range(12):
        r = int(rng.integers(st.num_requests))
        i = int(rng.integers(int(st.chunk_len[r])))
        h = int(rng.integers(cache.num_heads))
        wo, wl = _brute_row(cache, kp, vp, st, r, i, h)
        row = int(st.cu_chunk[r]) + i
        assert np.allclose(out[row, h], wo, rtol=0, atol=1e-12)
        assert lse[row, h] == pytest.approx(wl, abs=1e-12)
    # the sampled-row entry point is the same function
    so, sl = O.attention_rows(cache, kp, vp, st, [(0, 0, 1), (2, int(st.chunk_len[2]) - 1, 0)])
    assert np.array_equal(so[0], out[int(st.cu_chunk[0]), 1])
    assert np.array_equal(so[1], out[int(st.cu_chunk[3]) - 1, 0])
    assert sl[0] == lse[int(st.cu_chunk[0]), 1]


# ----------------------------------------------------------------------------
# grouped query heads and token trees (extensions; the paper's models have one K/V head per query head, Sec. 4.1,
# and HAT's own drafts are linear, Sec. 3.4; trees are the U-Medusa comparison system's, Sec. 4.1)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("group,tree", [(4, False), (1, True), (2, True)])
def test_brute_force_rows_grouped_heads_and_trees(group, tree):
    sc = W.mixed_13b(num_prefill=1, prefill_chunk=20, max_prefill_prefix=40, num_verify=3, draft=7,
                     min_verify_prefix=0, max_verify_prefix=50, H=2, d=64, seed=16, q_group=group, tree=tree)
    cache, st = sc.cache, sc.steps[0]
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(cache, kp, vp, st)
    out, lse = O.chunk_attention(cache, kp, vp, st)
    assert out.shape == (st.total_rows, 2 * group, 64)
    for r in range(st.num_requests):
        for i in range(0, int(st.chunk_len[r]), 3):
            for h in range(2 * group):
                wo, wl = _brute_row(cache, kp, vp, st, r, i, h)
                row = int(st.cu_chunk[r]) + i
                assert np.allclose(out[row, h], wo, rtol=0, atol=1e-12)
                assert lse[row, h] == pytest.approx(wl, abs=1e-12)


def test_grouped_heads_equal_repeated_kv_heads():
    """G query heads per K/V head == ordinary attention over a cache whose heads are each repeated G times."""
    G, H, d = 3, 2, 64
    sc = W.spec_verify(num_requests=3, min_prefix=5, max_prefix=60, max_draft=6, H=H, d=d, seed=17, q_group=G)
    cache, st = sc.cache, sc.steps[0]
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(cache, kp, vp, st)
    out, lse = O.chunk_attention(cache, kp, vp, st)
    wide = W.CacheSpec(cache.dtype, H * G, d, cache.num_pages, "paged")
    def widen_pool(pool):
        x = pool.reshape(cache.num_pages, H, cache.page_size, d)
        return np.ascontiguousarray(np.repeat(x, G, axis=1)).ravel()
    out2, lse2 = O.chunk_attention(wide, widen_pool(kp), widen_pool(vp), st)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_causal_tree_mask_is_the_default_and_a_path_is_a_linear_draft():
    sc = W.spec_verify(num_requests=4, min_prefix=0, max_prefix=40, max_draft=8, H=2, d=64, seed=18)
    cache, st = sc.cache, sc.steps[0]
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(cache, kp, vp, st)
    out, lse = O.chunk_attention(cache, kp, vp, st)
    # (1) the lower-triangular words reproduce the causal rule bit for bit
    st.tree_mask = np.concatenate([[(2 << i) - 1 for i in range(int(c))] for c in st.chunk_len]).astype(np.uint32)
    out_t, lse_t = O.chunk_attention(cache, kp, vp, st)
    assert np.array_equal(out, out_t) and np.array_equal(lse, lse_t)
    # (2) a random tree: every node's row equals the last row of the LINEAR draft made of its root-to-node path
    st.tree_mask = W.random_tree_masks(5, st.chunk_len)
    out_t, lse_t = O.chunk_attention(cache, kp, vp, st)
    kn = st.k_new.reshape(st.total_rows, -1); vn = st.v_new.reshape(st.total_rows, -1)
    for r in range(st.num_requests):
        P, Cn, base = int(st.prefix_len[r]), int(st.chunk_len[r]), int(st.cu_chunk[r])
        for i in range(Cn):
            path = [c for c in range(Cn) if (int(st.tree_mask[base + i]) >> c) & 1]
            assert path[-1] == i
            rows = [base + c for c in path]
            lin = types.SimpleNamespace(prefix_len=np.asarray([P], np.int32), chunk_len=np.asarray([len(path)], np.int32),
                                        cu_chunk=np.asarray([0, len(path)], np.int32),
                                        block_table=st.block_table[r:r + 1], q=st.q[rows], k_new=st.k_new[rows],
                                        v_new=st.v_new[rows])
            kp2, vp2 = kp.copy(), vp.copy()
            O.kv_append(cache, kp2, vp2, lin)          # the path's K/V at positions P .. P+len-1
            out_l, lse_l = O.chunk_attention(cache, kp2, vp2, lin)
            assert np.allclose(out_t[base + i], out_l[-1], rtol=0, atol=1e-13)
            assert np.allclose(lse_t[base + i], lse_l[-1], rtol=0, atol=1e-13)
    # (3) a word without any chunk bit at an empty prefix sees nothing
    st0 = _step([0], [2], st.block_table[:1], st.q[:2], st.k_new[:2], st.v_new[:2])
    st0.tree_mask = np.asarray([0, 2], np.uint32)
    o0, l0 = O.chunk_attention(cache, kp, vp, st0)
    assert np.all(o0[0] == 0) and np.all(l0[0] == -np.inf) and np.all(np.isfinite(l0[1]))


# ----------------------------------------------------------------------------
# library cross-check on the dense special case (full-prompt causal attention)
# ----------------------------------------------------------------------------
def _full_prompt_reference(qf, kf, vf):
    import torch
    q = torch.from_numpy(qf).permute(1, 0, 2)[None]      # [1,H,n,d]
    k = torch.from_numpy(kf).permute(1, 0, 2)[None]
    v = torch.from_numpy(vf).permute(1, 0, 2)[None]
    n = q.shape[2]
    mask = torch.ones(n, n, dtype=torch.bool).tril()
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask)
    return o[0].permute(1, 0, 2).numpy()                  # [n,H,d]


def _run_chunked(dtype, H, d, n, sizes, qb, kb, vb, layout="contiguous", table=None, num_pages=None):
    """Feed a prompt through the oracle as successive chunks of the given sizes."""
    num_pages = num_pages or (n + 15) // 16
    table = np.arange(num_pages)[None, :] if table is None else table
    cache = _cache(dtype, H, d, num_pages, layout)
    kp = W.normal_bits(cache.pool_elems, dtype, 99)       # stale garbage everywhere
    vp = W.normal_bits(cache.pool_elems, dtype, 98)
    outs, lses, p = [], [], 0
    for c in sizes:
        st = _step([p], [c], table, qb[p:p + c], kb[p:p + c], vb[p:p + c])
        O.kv_append(cache, kp, vp, st)
        o, l = O.chunk_attention(cache, kp, vp, st)
        outs.append(o); lses.append(l); p += c
    assert p == n
    return np.concatenate(outs), np.concatenate(lses)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_chunked_equals_full_prompt_and_library_sdpa(dtype):
    # Sec. 2.1 / 3.3: a prompt fed as chunks over several steps gives what one-shot prefill gives.
    H, d, n = 2, 64, 100
    qb = W.normal_bits(n * H * d, dtype, 1).reshape(n, H, d)
    kb = W.normal_bits(n * H * d, dtype, 2).reshape(n, H, d)
    vb = W.normal_bits(n * H * d, dtype, 3).reshape(n, H, d)
    ref = _full_prompt_reference(W.bits_to_f64(qb, dtype), W.bits_to_f64(kb, dtype), W.bits_to_f64(vb, dtype))
    whole, whole_lse = _run_chunked(dtype, H, d, n, [n], qb, kb, vb)
    assert np.allclose(whole, ref, rtol=0, atol=1e-12)
    for sizes in ([1] * n, [7] * 14 + [2], [16] * 6 + [4], [64, 36], [3, 50, 47]):
        o, l = _run_chunked(dtype, H, d, n, sizes, qb, kb, vb)
        assert np.array_equal(o, whole), sizes            # same keys in the same order: bit-identical
        assert np.array_equal(l, whole_lse), sizes
    # lse against logsumexp of the dense score matrix
    Q, K = W.bits_to_f64(qb, dtype), W.bits_to_f64(kb, dtype)
    S = np.einsum("ihc,jhc->hij", Q, K) / math.sqrt(d)
    for i in (0, 1, 57, n - 1):
        want = np.log(np.exp(S[:, i, :i + 1] - S[:, i, :i + 1].max(-1, keepdims=True)).sum(-1)) + S[:, i, :i + 1].max(-1)
        assert np.allclose(whole_lse[i], want, rtol=0, atol=1e-12)


def test_draft_verification_equals_sequential_decode():
    # Sec. 2.1 / 3.4: verifying k drafts in one step == k single-token decode steps.
    H, d, P, k = 2, 64, 37, 6
    n = P + k
    qb = W.normal_bits(n * H * d, "fp16", 21).reshape(n, H, d)
    kb = W.normal_bits(n * H * d, "fp16", 22).reshape(n, H, d)
    vb = W.normal_bits(n * H * d, "fp16", 23).reshape(n, H, d)
    one_step, l1 = _run_chunked("fp16", H, d, n, [P, k], qb, kb, vb)
    seq, l2 = _run_chunked("fp16", H, d, n, [P] + [1] * k, qb, kb, vb)
    assert np.array_equal(one_step, seq) and np.array_equal(l1, l2)


def test_page_permutation_and_layout_invariance():
    H, d, n = 2, 64, 75
    qb = W.normal_bits(n * H * d, "fp16", 31).reshape(n, H, d)
    kb = W.normal_bits(n * H * d, "fp16", 32).reshape(n, H, d)
    vb = W.normal_bits(n * H * d, "fp16", 33).reshape(n, H, d)
    base, base_l = _run_chunked("fp16", H, d, n, [40, 35], qb, kb, vb)
    rng = np.random.default_rng(2)
    for layout in ("contiguous", "paged"):
        perm = rng.permutation(9)[:5][None, :]            # 5 of 9 pages, shuffled
        o, l = _run_chunked("fp16", H, d, n, [40, 35], qb, kb, vb, layout=layout, table=perm, num_pages=9)
        assert np.array_equal(o, base) and np.array_equal(l, base_l)


# ----------------------------------------------------------------------------
# log-sum-exp: split/merge identity and shift invariance
# ----------------------------------------------------------------------------
def test_split_merge_identity():
    sc = W.spec_verify(num_requests=2, min_prefix=40, max_prefix=90, max_draft=5, H=2, d=64, seed=8)
    cache, st = sc.cache, sc.steps[0]
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(cache, kp, vp, st)
    out, lse = O.chunk_attention(cache, kp, vp, st)
    for r in range(2):
        i = int(st.chunk_len[r]) - 1
        n = int(st.prefix_len[r]) + i + 1
        for cuts in ([0, 17, n], [0, 1, 33, 34, n], [0, n, n + 5]):     # last part is empty
            parts = [(r, i, 1, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
            po, pl = O.attention_rows(cache, kp, vp, st, parts)
            mo, ml = O.merge(po, pl)
            row = int(st.cu_chunk[r]) + i
            assert np.allclose(mo, out[row, 1], rtol=0, atol=1e-13)
            assert ml == pytest.approx(lse[row, 1], abs=1e-13)


def test_merge_closed_form():
    # two parts with lse = ln 1 and ln 3 => weights 1/4 and 3/4, lse = ln 4
    o, l = O.merge(np.array([[4.0, 0.0], [0.0, 8.0]]), np.array([0.0, math.log(3.0)]))
    assert np.allclose(o, [1.0, 6.0], rtol=0, atol=1e-15)
    assert l == pytest.approx(math.log(4.0), abs=1e-15)
    o, l = O.merge(np.array([[1.0, 2.0], [9.0, 9.0]]), np.array([-0.5, -np.inf]))
    assert np.array_equal(o, [1.0, 2.0]) and l == -0.5


def test_score_shift_moves_lse_only():
    # Last feature: q = a, every key = b  => every score gains a*b/sqrt(d).
    H, d, n = 1, 64, 50
    rng = np.random.default_rng(9)
    k = rng.standard_normal((n, H, d)).astype(np.float32)
    v = rng.standard_normal((n, H, d)).astype(np.float32)
    q = rng.standard_normal((1, H, d)).astype(np.float32)
    q[..., -1] = 4.0
    res = []
    for b in (0.0, 2.0):
        k[..., -1] = b
        cache = _cache("fp16", H, d, 4, "contiguous")
        kp = np.zeros(cache.pool_elems, np.uint16); vp = np.zeros(cache.pool_elems, np.uint16)
        kp[:n * H * d] = _bits(k).ravel(); vp[:n * H * d] = _bits(v).ravel()
        st = _step([n - 1], [1], [[0, 1, 2, 3]], _bits(q), _bits(k[-1:]), _bits(v[-1:]))
        res.append(O.chunk_attention(cache, kp, vp, st))
    assert np.allclose(res[0][0], res[1][0], rtol=0, atol=1e-13)
    assert res[1][1][0, 0] - res[0][1][0, 0] == pytest.approx(4.0 * 2.0 / 8.0, abs=1e-12)


def test_explicit_scale_argument():
    sc = W.tiny(prompt=32, chunk=32, draft=2, H=2, d=64, seed=13)
    cache, st = sc.cache, sc.steps[0]
    a, la = O.chunk_attention(cache, sc.k_pool, sc.v_pool, st)
    b, lb = O.chunk_attention(cache, sc.k_pool, sc.v_pool, st, sm_scale=0.125)
    assert np.array_equal(a, b) and np.array_equal(la, lb)
    c, _ = O.chunk_attention(cache, sc.k_pool, sc.v_pool, st, sm_scale=0.0)    # uniform weights
    V = W.bits_to_f64(sc.v_pool, "fp16").reshape(-1, 2, 64)
    assert np.allclose(c[9], V[:10].mean(0), rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------
# append: bit-exact placement, untouched slots, rollback
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("layout", ["paged", "contiguous"])
def test_append_placement_and_untouched_slots(layout):
    H, d = 3, 64
    cache = _cache("fp16", H, d, 7, layout)
    rng = np.random.default_rng(12)
    kp = rng.integers(0, 65536, cache.pool_elems).astype(np.uint16)
    vp = rng.integers(0, 65536, cache.pool_elems).astype(np.uint16)
    k0, v0 = kp.copy(), vp.copy()
    table = [[5, 2, 6], [3, 0, -1]]
    prefix, chunk = [13, 16], [21, 9]                      # mid-page start; page-aligned start
    T = sum(chunk)
    kn = rng.integers(0, 65536, (T, H, d)).astype(np.uint16)
    vn = rng.integers(0, 65536, (T, H, d)).astype(np.uint16)
    O.kv_append(cache, kp, vp, _step(prefix, chunk, table, kn, kn, vn))
    shape = (7, H, 16, d) if layout == "paged" else (7, 16, H, d)
    K, V, K0 = kp.reshape(shape), vp.reshape(shape), k0.reshape(shape)
    touched = np.zeros(shape[:3], bool)
    row = 0
    for r in range(2):
        for i in range(chunk[r]):
            p = prefix[r] + i
            page, slot = table[r][p // 16], p % 16
            for h in range(H):
                idx = (page, h, slot) if layout == "paged" else (page, slot, h)
                assert np.array_equal(K[idx], kn[row, h]) and np.array_equal(V[idx], vn[row, h])
                touched[idx] = True
            row += 1
    assert np.array_equal(K[~touched], K0[~touched])
    assert np.array_equal(vp.reshape(shape)[~touched], v0.reshape(shape)[~touched])
    assert touched.sum() == T * H


def test_rollback_overwrites_rejected_drafts():
    # Sec. 3.4: after a round accepts 3 of 8 drafts the next chunk restarts at prefix+3.
    H, d = 2, 64
    cache = _cache("fp16", H, d, 3, "paged")
    kp = np.zeros(cache.pool_elems, np.uint16); vp = np.zeros(cache.pool_elems, np.uint16)
    table = [[2, 0, 1]]
    first = np.arange(8 * H * d, dtype=np.uint16).reshape(8, H, d) + 1000
    second = np.arange(5 * H * d, dtype=np.uint16).reshape(5, H, d) + 30000
    O.kv_append(cache, kp, vp, _step([10], [8], table, first, first, first))
    O.kv_append(cache, kp, vp, _step([13], [5], table, second, second, second))
    K = kp.reshape(3, H, 16, d)
    for p in range(10, 18):
        page, slot = table[0][p // 16], p % 16
        want = first[p - 10] if p < 13 else second[p - 13]
        assert np.array_equal(K[page, :, slot, :], want)
    assert not K[table[0][0], :, :10].any()
