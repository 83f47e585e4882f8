"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element on reduced
sizes of the five workloads, on sampled rows at their full sizes, and on the edge cases."""
import types

import numpy as np
import pytest

from oracle import hat_oracle as O
from paper_2503_18989_b200 import workloads as W

from common import assert_parity, oracle_replay

pytestmark = pytest.mark.gpu


def _run(sc, device, fused_append=True):
    from paper_2503_18989_b200 import runner
    return runner.run_scenario(sc, device, fused_append=fused_append)


def _check_full(sc, device, fused_append=True):
    """Every element of out/lse of every step, and both pools bit for bit."""
    cache, got = _run(sc, device, fused_append)
    kp, vp, want = oracle_replay(sc)
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, kp), "K pool differs from the oracle's append"
    assert np.array_equal(gv, vp), "V pool differs from the oracle's append"
    for s, ((go, gl), (wo, wl)) in enumerate(zip(got, want)):
        assert_parity(go, wo, f"{sc.name} step {s} out")
        assert_parity(gl, wl, f"{sc.name} step {s} lse")
    return got, want


def _check_sampled(sc, device, num_samples=400, seed=0):
    """Full-size run: pools bit for bit; out/lse on sampled (request, row, head) triples, always
    including the first and last row of every request."""
    cache, got = _run(sc, device)
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    rng = np.random.default_rng(seed)
    for s, st in enumerate(sc.steps):
        O.kv_append(sc.cache, kp, vp, st)
        samples = []
        live = [r for r in range(st.num_requests) if st.chunk_len[r] > 0]
        for r in live:
            for i in {0, int(st.chunk_len[r]) - 1}:
                samples.append((r, i, int(rng.integers(sc.cache.num_heads))))
        while len(samples) < num_samples // len(sc.steps):
            r = live[int(rng.integers(len(live)))]
            samples.append((r, int(rng.integers(st.chunk_len[r])), int(rng.integers(sc.cache.num_heads))))
        samples = np.asarray(samples, np.int64)
        wo, wl = O.attention_rows(sc.cache, kp, vp, st, samples)
        rows = st.cu_chunk[samples[:, 0]] + samples[:, 1]
        go = got[s][0][rows, samples[:, 2]]
        gl = got[s][1][rows, samples[:, 2]]
        assert_parity(go, wo, f"{sc.name} step {s} sampled out")
        assert_parity(gl, wl, f"{sc.name} step {s} sampled lse")
        assert np.isfinite(got[s][0]).all() and np.isfinite(got[s][1]).all()
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, kp) and np.array_equal(gv, vp)


# ----------------------------------------------------------------------------
# the five workloads: reduced sizes, every element
# ----------------------------------------------------------------------------
def test_tiny_every_element(cuda_device):
    _check_full(W.tiny(), cuda_device)                       # the full "tiny" configuration


def test_head_dim_64_chunks_run_on_the_tcgen05_kernel(cuda_device):
    """The 64-row chunks of the tiny configuration (8 heads x 64) take the tcgen05 tile kernel, not the mma.sync one."""
    from paper_2503_18989_b200 import runner
    sc = W.tiny()
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert sc.cache.head_dim == 64 and ds.info["num_prefill_requests"] == 1 and ds.info["prefill_kernel"] == 1
    ds.close()


def test_llama7b_chunked_reduced(cuda_device):
    _check_full(W.llama7b_chunked(prompt=640, chunk=256, H=4), cuda_device)   # 256, 256, ragged 128


def test_ragged_prefill_reduced(cuda_device):
    _check_full(W.ragged_prefill(num_requests=7, max_prefix=640, H=3), cuda_device)


def test_spec_verify_reduced(cuda_device):
    _check_full(W.spec_verify(num_requests=9, min_prefix=100, max_prefix=1500, H=5), cuda_device)


def test_mixed_13b_reduced(cuda_device):
    _check_full(W.mixed_13b(num_prefill=2, prefill_chunk=512, max_prefill_prefix=700, num_verify=6,
                            min_verify_prefix=200, max_verify_prefix=1200, H=3), cuda_device)


# ----------------------------------------------------------------------------
# the five workloads: full sizes, sampled rows
# ----------------------------------------------------------------------------
def test_llama7b_chunked_full_size_sampled(cuda_device):
    _check_sampled(W.llama7b_chunked(), cuda_device, num_samples=480)


def test_ragged_prefill_full_size_sampled(cuda_device):
    _check_sampled(W.ragged_prefill(), cuda_device)


def test_spec_verify_full_size_sampled(cuda_device):
    _check_sampled(W.spec_verify(), cuda_device)


def test_mixed_13b_full_size_sampled(cuda_device):
    _check_sampled(W.mixed_13b(), cuda_device)


# ----------------------------------------------------------------------------
# variants and edge cases
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,layout", [("bf16", 128, "paged"), ("fp16", 64, "paged"), ("bf16", 64, "contiguous"),
                                           ("fp16", 128, "contiguous")])
def test_dtype_headdim_layout_variants(cuda_device, dtype, d, layout):
    sc = W.ragged_prefill(num_requests=4, max_prefix=300, chunk_choices=(17, 40, 64, 130), H=2, d=d, dtype=dtype,
                          seed=77)
    if layout == "contiguous":
        sc.cache.layout = "contiguous"                       # same pool bits, different strides
    _check_full(sc, cuda_device)
    sc = W.spec_verify(num_requests=4, min_prefix=1, max_prefix=400, max_draft=16, H=2, d=d, dtype=dtype, seed=78)
    if layout == "contiguous":
        sc.cache.layout = "contiguous"
    _check_full(sc, cuda_device)


def _manual(dtype, H, d, prefix, chunk, seed, num_pages=None, table=None, layout="paged", q_group=1, tree=False):
    """Batch with hand-picked prefix/chunk lengths (H K/V heads, H * q_group query heads)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if table is None:
        table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=5)
    st = W._make_step(seed + 100, dtype, H, d, prefix, chunk, table, q_heads=H * q_group)
    if tree:
        st.tree_mask = W.random_tree_masks(seed + 200, chunk)
    return W._scenario("manual", dtype, H, d, layout, num_pages, [st], seed + 100)


def test_every_chunk_length_class_and_ragged_tails(cuda_device):
    # 0 (no-op), 1 at an empty cache, 8, 16 (largest streaming), 17 (smallest tile), one short of and one past
    # a tile, prefix not a multiple of the page size for a tile-class chunk
    prefix = [40, 0, 33, 250, 5, 100, 77, 0, 1023]
    chunk = [0, 1, 8, 16, 17, 63, 65, 129, 7]
    _check_full(_manual("fp16", 2, 128, prefix, chunk, 5), cuda_device)
    _check_full(_manual("bf16", 2, 64, prefix, chunk, 6), cuda_device)


def test_empty_batch_and_all_zero_chunks(cuda_device):
    from paper_2503_18989_b200 import binding as B, runner
    sc = _manual("fp16", 2, 128, [10, 20], [0, 0], 9)
    cache, got = _run(sc, cuda_device)
    assert got[0][0].shape == (0, 2, 128)
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, sc.k_pool) and np.array_equal(gv, sc.v_pool)
    plan = B.hat_plan_create(cache.desc, 2, np.zeros(1, np.int32), np.zeros(0, np.int32), np.zeros(0, np.int32),
                             np.zeros((0, 0), np.int32))
    B.hat_chunk_attention(cache.desc, plan, None, None, None, None, None)      # valid no-op
    B.hat_kv_append(cache.desc, plan, None, None)


def test_separate_append_equals_fused_append(cuda_device):
    sc = W.mixed_13b(num_prefill=1, prefill_chunk=96, max_prefill_prefix=200, num_verify=3, min_verify_prefix=20,
                     max_verify_prefix=300, H=2, seed=31)
    c1, r1 = _run(sc, cuda_device, fused_append=True)
    c2, r2 = _run(sc, cuda_device, fused_append=False)
    for a, b in zip(c1.pools_to_host(), c2.pools_to_host()):
        assert np.array_equal(a, b)
    assert np.array_equal(r1[0][0], r2[0][0]) and np.array_equal(r1[0][1], r2[0][1])
    # and running the same call twice gives the same bits
    c3, r3 = _run(sc, cuda_device, fused_append=True)
    assert np.array_equal(r1[0][0], r3[0][0]) and np.array_equal(r1[0][1], r3[0][1])


def test_many_key_ranges_per_request(cuda_device):
    # one long request alone in the batch: the scheduler cuts it into the maximum number of ranges
    sc = _manual("fp16", 1, 128, [9000], [3], 12)
    from paper_2503_18989_b200 import binding as B
    got, want = _check_full(sc, cuda_device)


def test_rollback_then_verify_again(cuda_device):
    # Sec. 3.4: 6 drafts sent, 2 accepted; the next round restarts at prefix+2 and overwrites the rest.
    H, d, P = 2, 128, 45
    rng = np.random.Generator(np.random.PCG64(3))
    table, num_pages = W._place_pages(rng, [P + 20], slack_pages=3)
    s1 = W._make_step(500, "fp16", H, d, [P], [6], table)
    s2 = W._make_step(600, "fp16", H, d, [P + 2], [5], table)
    sc = W._scenario("rollback", "fp16", H, d, "paged", num_pages, [s1, s2], 700)
    _check_full(sc, cuda_device)


def test_explicit_scale_and_stale_nan_slots(cuda_device):
    from paper_2503_18989_b200 import runner
    sc = _manual("fp16", 2, 128, [37, 200], [4, 70], 15)
    st = sc.steps[0]
    # poison every slot the batch must not read: beyond prefix+chunk in the last page, and unowned pages
    owned = np.zeros(sc.cache.num_pages, bool)
    K = sc.k_pool.reshape(sc.cache.num_pages, 2, 16, 128); V = sc.v_pool.reshape(K.shape)
    for r in range(2):
        n = int(st.prefix_len[r] + st.chunk_len[r])
        pages = st.block_table[r][: (n + 15) // 16]
        owned[pages] = True
        if n % 16:
            K[pages[-1], :, n % 16:, :] = 0x7E00           # fp16 NaN
            V[pages[-1], :, n % 16:, :] = 0x7E00
    K[~owned] = 0x7E00; V[~owned] = 0x7E00
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    ds.attend(fused_append=True, sm_scale=0.05)
    go, gl = ds.results()
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, st)
    wo, wl = O.chunk_attention(sc.cache, kp, vp, st, sm_scale=float(np.float32(0.05)))
    assert_parity(go, wo, "scaled out"); assert_parity(gl, wl, "scaled lse")


def test_launch_errors_are_reported_before_any_work(cuda_device):
    from paper_2503_18989_b200 import binding as B, runner
    sc = W.spec_verify(num_requests=2, min_prefix=600, max_prefix=900, H=2, seed=41)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.workspace_bytes > 0
    with pytest.raises(B.HatError) as e:
        B.hat_chunk_attention(cache.desc, ds.plan, ds.q, None, None, ds.out, ds.lse, 0.0, ds.workspace, 16)
    assert e.value.status == B.HAT_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(B.HatError) as e:
        B.hat_chunk_attention(cache.desc, ds.plan, ds.q, ds.k_new, None, ds.out, ds.lse, 0.0, ds.workspace,
                              ds.workspace_bytes)
    assert e.value.status == B.HAT_ERR_INVALID_ARG
    with pytest.raises(B.HatError) as e:
        B.hat_chunk_attention(cache.desc, ds.plan, None, None, None, ds.out, ds.lse, 0.0, ds.workspace,
                              ds.workspace_bytes)
    assert e.value.status == B.HAT_ERR_INVALID_ARG
    other = B.make_cache_desc("bf16", sc.cache.num_pages, 2, 128, sc.cache.stride_page, sc.cache.stride_token,
                              sc.cache.stride_head, cache.k, cache.v)
    with pytest.raises(B.HatError) as e:
        B.hat_kv_append(other, ds.plan, ds.k_new, ds.v_new)
    assert e.value.status == B.HAT_ERR_INVALID_ARG
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, sc.k_pool) and np.array_equal(gv, sc.v_pool)     # nothing was written
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK


def test_host_buffer_entry_point(cuda_device):
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    sc = W.mixed_13b(num_prefill=1, prefill_chunk=80, max_prefill_prefix=150, num_verify=2, min_verify_prefix=30,
                     max_verify_prefix=700, H=2, seed=51)
    st = sc.steps[0]
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    T, H, d = st.total_rows, 2, 128
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    q, k, v = pin(st.q), pin(st.k_new), pin(st.v_new)
    out = torch.empty((T, H, d), dtype=torch.float32).pin_memory()
    lse = torch.empty((T, H), dtype=torch.float32).pin_memory()
    nbytes = B.hat_plan_staging_bytes(ds.plan)
    staging = torch.empty(nbytes, dtype=torch.uint8, device=cuda_device)
    B.hat_chunk_attention_host(cache.desc, ds.plan, q, k, v, out, lse, 0.0, staging, nbytes, ds.workspace,
                               ds.workspace_bytes)
    torch.cuda.synchronize()
    kp, vp, want = oracle_replay(sc)
    assert_parity(out.numpy(), want[0][0], "host entry out")
    assert_parity(lse.numpy(), want[0][1], "host entry lse")
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
    # two steps in flight, as the benchmark's end-to-end leg runs them: alternate streams, each with its own staging
    # and result buffers; the copies of one overlap the other's kernels, the plan keeps the kernels in order
    streams = [torch.cuda.Stream(cuda_device), torch.cuda.Stream(cuda_device)]
    outs = [(torch.full((T, H, d), float("nan"), dtype=torch.float32).pin_memory(),
             torch.full((T, H), float("nan"), dtype=torch.float32).pin_memory(),
             torch.empty(nbytes, dtype=torch.uint8, device=cuda_device)) for _ in streams]
    for i in range(6):
        o, l, stg = outs[i % 2]
        B.hat_chunk_attention_host(cache.desc, ds.plan, q, k, v, o, l, 0.0, stg, nbytes, ds.workspace,
                                   ds.workspace_bytes, streams[i % 2].cuda_stream)
    torch.cuda.synchronize()
    for o, l, _ in outs:
        assert_parity(o.numpy(), want[0][0], "host entry, two in flight, out")
        assert_parity(l.numpy(), want[0][1], "host entry, two in flight, lse")


@pytest.mark.parametrize("kernel,code", [("tc5", 1), ("pair", 3)])
def test_bounded_wait_gives_up_and_the_context_stays_usable(cuda_device, kernel, code, monkeypatch):
    """Failure detection without a fault: the tile kernel's producer withholds one transfer, the waiting
    warps give up after the (shortened) bound (in the CTA-pair kernel both CTAs of every pair), the status word
    reports it, and the next call is correct."""
    from paper_2503_18989_b200 import binding as B, runner
    monkeypatch.setenv("HAT_PREFILL_KERNEL", kernel)
    sc = _manual("fp16", 2, 128, [300], [200], 21)
    st = sc.steps[0]
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    assert ds.info["prefill_kernel"] == code
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    B.hat_plan_set_wait_limit(ds.plan, 20_000_000, withhold_next_call=True)      # about 10 ms
    ds.attend(fused_append=True)
    assert B.hat_last_device_status(ds.plan) == B.HAT_ERR_DEVICE_TIMEOUT
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK                            # reading clears the word
    B.hat_plan_set_wait_limit(ds.plan, 0)
    ds.attend(fused_append=True)                                                    # the self test was one-shot
    go, gl = ds.results()
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    kp, vp, want = oracle_replay(sc)
    assert_parity(go, want[0][0], "out after a timed-out call")
    assert_parity(gl, want[0][1], "lse after a timed-out call")


def test_long_prefill_request_is_cut_into_at_most_32_key_ranges(cuda_device):
    from paper_2503_18989_b200 import binding as B, runner
    sc = _manual("fp16", 1, 128, [20000], [300], 22)
    cache, got = _run(sc, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert 1 < ds.info["max_splits"] <= 32 and ds.info["num_merge_rows"] == 300
    rng = np.random.default_rng(0)
    samples = np.asarray([(0, int(i), 0) for i in [0, 127, 128, 255, 256, 299, *rng.integers(0, 300, 20)]], np.int64)
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, sc.steps[0])
    wo, wl = O.attention_rows(sc.cache, kp, vp, sc.steps[0], samples)
    assert_parity(got[0][0][samples[:, 1], 0], wo, "long prefill out")
    assert_parity(got[0][1][samples[:, 1], 0], wl, "long prefill lse")


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_key_ranges_that_only_the_second_query_tile_sees(cuda_device, dtype, monkeypatch):
    """Ranges of 256 keys over 256-row units whose prefix is 128 past a multiple of 256: the last range of every
    unit lies wholly behind the first query tile's last row, so that tile has no work in it while the second
    one has; with 2 heads and 120 requests every CTA of the persistent kernel strings several such units
    between ordinary ones."""
    monkeypatch.setenv("HAT_PREFILL_SPLIT_LEN", "256")
    prefix = [128 + 256 * (r % 4) for r in range(120)]
    chunk = [256 if r % 5 else 200 for r in range(120)]
    sc = _manual(dtype, 2, 128, prefix, chunk, 23)
    from paper_2503_18989_b200 import runner
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.info["prefill_kernel"] in (1, 3) and ds.info["prefill_split_len"] == 256 and ds.info["max_splits"] == 5
    _check_full(sc, cuda_device)


@pytest.mark.parametrize("seed", range(12))
def test_random_small_batches(cuda_device, seed):
    """Seeded random batches that mix every chunk class, odd prefixes, both types, both head sizes and both
    layouts, with few heads so that the persistent tile kernel strings several units through one CTA and
    key ranges get cut (few CTAs)."""
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    dtype = ["fp16", "bf16"][seed % 2]
    d = [128, 128, 64][seed % 3]
    H = int(rng.integers(1, 4))
    R = int(rng.integers(1, 9))
    kinds = rng.integers(0, 5, size=R)
    chunk = np.where(kinds == 0, rng.integers(0, 3, size=R),                 # empty / one or two rows
            np.where(kinds == 1, rng.integers(1, 17, size=R),                # streaming class
            np.where(kinds == 2, rng.integers(17, 130, size=R),              # one query tile
            np.where(kinds == 3, rng.integers(130, 300, size=R),             # two query tiles, ragged
                     rng.integers(300, 700, size=R)))))                      # several 256-row items
    prefix = np.where(rng.random(R) < 0.3, 0, rng.integers(0, 1500, size=R))
    sc = _manual(dtype, H, d, prefix, chunk, 2000 + seed, layout=["paged", "contiguous"][(seed // 2) % 2])
    _check_full(sc, cuda_device, fused_append=bool(seed % 2))


def test_verify_rows_are_final_before_the_prompt_chunks_run(cuda_device):
    """Decode-phase requests of a mixed batch are not held back by its prompt chunks: the plan's event fires
    after the streaming kernel, well before the whole call has finished (Sec. 2.1 / 3.3)."""
    import time
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    sc = W.mixed_13b(num_prefill=6, prefill_chunk=512, max_prefill_prefix=6000, num_verify=8, min_verify_prefix=256,
                     max_verify_prefix=1024, H=16, seed=61)
    st = sc.steps[0]
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    assert B.hat_plan_verify_event(ds.plan)
    for _ in range(3):
        ds.attend()
    torch.cuda.synchronize()
    best = 1.0
    for _ in range(5):
        t0 = time.perf_counter()
        ds.attend()
        B.hat_plan_wait_verify(ds.plan)
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        best = min(best, (t1 - t0) / (t2 - t0))
    assert best < 0.6, f"verify rows became final only after {best:.2f} of the call"
    # and the rows are right (whole batch against the oracle)
    go, gl = ds.results()
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    O.kv_append(sc.cache, kp, vp, st)
    short = [r for r in range(st.num_requests) if st.chunk_len[r] <= 16]
    samples = np.asarray([(r, i, h) for r in short for i in range(int(st.chunk_len[r])) for h in (0, 15)], np.int64)
    wo, wl = O.attention_rows(sc.cache, kp, vp, st, samples)
    rows = st.cu_chunk[samples[:, 0]] + samples[:, 1]
    assert_parity(go[rows, samples[:, 2]], wo, "verify rows out")
    assert_parity(gl[rows, samples[:, 2]], wl, "verify rows lse")


# ----------------------------------------------------------------------------
# grouped query heads and token trees
# ----------------------------------------------------------------------------
_GQA_PREFIX = [40, 0, 33, 250, 5, 1000, 77, 0, 1023, 600, 17]
_GQA_CHUNK = [0, 1, 8, 16, 17, 3, 65, 129, 7, 300, 12]


@pytest.mark.parametrize("dtype,d,group,layout", [("fp16", 128, 2, "paged"), ("bf16", 128, 4, "paged"),
                                                  ("fp16", 64, 8, "paged"), ("bf16", 64, 3, "contiguous"),
                                                  ("fp16", 128, 5, "contiguous")])
def test_grouped_query_heads(cuda_device, dtype, d, group, layout):
    """G query heads share each K/V head: every chunk class, chunk rows x G both below and above one 16-row
    slab, q / out / lse with G times the heads of the pools."""
    sc = _manual(dtype, 2, d, _GQA_PREFIX, _GQA_CHUNK, 31 + group, layout=layout, q_group=group)
    got, want = _check_full(sc, cuda_device)
    assert got[0][0].shape == (sum(_GQA_CHUNK), 2 * group, d)


@pytest.mark.parametrize("dtype,d,group", [("fp16", 128, 1), ("bf16", 128, 4), ("bf16", 64, 2)])
def test_token_trees(cuda_device, dtype, d, group):
    """Random token trees on every short chunk (1..16 rows, empty and mid-page prefixes, ranges cut by the
    scheduler), causal long chunks in the same batch."""
    sc = _manual(dtype, 2, d, _GQA_PREFIX + [9000], _GQA_CHUNK + [16], 41 + group, q_group=group, tree=True)
    st = sc.steps[0]
    assert any(int(w) != (2 << i) - 1 for r in range(st.num_requests) if st.chunk_len[r] <= 16
               for i, w in enumerate(st.tree_mask[st.cu_chunk[r]:st.cu_chunk[r + 1]])), "the trees must not all be chains"
    _check_full(sc, cuda_device)


def test_tree_row_that_sees_nothing_and_rows_that_see_later_positions(cuda_device):
    from paper_2503_18989_b200 import runner
    sc = _manual("fp16", 2, 128, [0, 20], [3, 4], 51, q_group=2)
    st = sc.steps[0]
    st.tree_mask = np.asarray([0b000, 0b110, 0b101, 0b1000, 0b0011, 0b1111, 0b0100], np.uint32)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    ds.attend()
    go, gl = ds.results()
    kp, vp, want = oracle_replay(sc)
    wo, wl = want[0]
    assert np.all(go[0] == 0) and np.all(gl[0] == -np.inf) and np.all(wl[0] == -np.inf)
    assert_parity(go[1:], wo[1:], "tree out")
    assert_parity(gl[1:], wl[1:], "tree lse")


@pytest.mark.parametrize("which", ["stream", "tile"])
def test_grouped_heads_and_trees_on_the_mma_sync_kernels(cuda_device, which, monkeypatch):
    monkeypatch.setenv("HAT_STREAM_KERNEL" if which == "stream" else "HAT_PREFILL_KERNEL", "mma")
    sc = _manual("bf16", 2, 128, _GQA_PREFIX, _GQA_CHUNK, 61, q_group=4, tree=True)
    _check_full(sc, cuda_device)


# ----------------------------------------------------------------------------
# output in the cache's 16-bit type
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,group", [("fp16", 128, 1), ("bf16", 128, 2), ("fp16", 64, 1), ("bf16", 64, 4)])
def test_sixteen_bit_output(cuda_device, dtype, d, group, monkeypatch):
    """hat_chunk_attention_out16: every kernel's final rows (streaming, tile, and rows merged from key ranges)
    equal the fp32 entry point's rows rounded to nearest, bit for bit where no fp32 value sits on a rounding
    boundary, and lie within the tolerance plus half a unit in the last place of the oracle's value."""
    from paper_2503_18989_b200 import runner
    monkeypatch.setenv("HAT_PREFILL_SPLIT_LEN", "256")           # some tile rows go through the merge kernel too
    sc = _manual(dtype, 2, d, _GQA_PREFIX + [9000], _GQA_CHUNK + [5], 71, q_group=group)
    st = sc.steps[0]
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, st)
    assert ds.info["num_merge_rows"] > 0
    ds.attend()
    o32, l32 = ds.results()
    ds.attend16(fused_append=False)
    import torch
    torch.cuda.synchronize()
    bits = ds.out16.cpu().numpy().view(np.uint16)
    got = W.bits_to_f64(bits, dtype)
    assert np.array_equal(ds.lse.cpu().numpy(), l32), "lse must not depend on the output type"
    want_bits = W.f32_to_bits(o32, dtype)
    exact = np.mean(bits == want_bits)
    assert exact > 0.999, f"only {exact:.4f} of the 16-bit outputs equal the rounded fp32 outputs"
    assert np.max(np.abs(bits.astype(np.int32) - want_bits.astype(np.int32))[np.isfinite(got)]) <= 1
    kp, vp, want = oracle_replay(sc)
    ref = want[0][0]
    ulp_half = np.abs(ref) * (2.0 ** -11 if dtype == "fp16" else 2.0 ** -8)
    err = np.abs(got - ref)
    from common import ABS_TOL
    assert np.all(err <= ABS_TOL + ulp_half), f"max excess {np.max(err - ulp_half):.3e}"


def test_mixed_batch_with_the_tile_kernel_on_a_side_stream(cuda_device, monkeypatch):
    """Optional throughput mode: the tile kernel starts on all but 56 SMs on a stream of the plan while the streaming
    kernel runs, and a second tile grid joins on the freed SMs; same results, also when called back to back."""
    from paper_2503_18989_b200 import runner
    monkeypatch.setenv("HAT_SIDE_SMS", "56")
    monkeypatch.setenv("HAT_PREFILL_KERNEL", "tc5")           # the mode exists for the one-CTA tile kernel
    sc = W.mixed_13b(num_prefill=5, prefill_chunk=384, max_prefill_prefix=3000, num_verify=12, min_verify_prefix=100,
                     max_verify_prefix=2000, H=4, seed=81)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.info["prefill_kernel"] == 1
    for _ in range(3):
        ds.attend()
    go, gl = ds.results()
    kp, vp, want = oracle_replay(sc)
    assert_parity(go, want[0][0], "side-stream out")
    assert_parity(gl, want[0][1], "side-stream lse")


def test_the_call_can_be_captured_in_a_cuda_graph_and_replayed(cuda_device):
    """hat_chunk_attention is stream-ordered and neither allocates nor synchronises, so a caller can capture the
    launch set of a step (append, streaming kernel, merge, tile kernel) once and replay it."""
    import torch
    from paper_2503_18989_b200 import runner
    sc = W.mixed_13b(num_prefill=3, prefill_chunk=300, max_prefill_prefix=5000, num_verify=6, min_verify_prefix=3000,
                     max_verify_prefix=9000, H=2, seed=91)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.info["num_merge_rows"] > 0
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(torch.cuda.current_stream(cuda_device))
    with torch.cuda.stream(side):
        ds.attend(stream=side.cuda_stream)                     # warm-up outside the capture
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ds.attend(stream=side.cuda_stream)
    torch.cuda.current_stream(cuda_device).wait_stream(side)
    ds.out.fill_(float("nan")); ds.lse.fill_(float("nan"))
    for _ in range(3):
        graph.replay()
    go, gl = ds.results()
    kp, vp, want = oracle_replay(sc)
    assert_parity(go, want[0][0], "graph replay out")
    assert_parity(gl, want[0][1], "graph replay lse")
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, kp) and np.array_equal(gv, vp)


def test_capture_on_another_stream_than_the_plans_earlier_calls(cuda_device):
    """Warm-up calls on one stream, then the same plan's call captured on another stream (ordered behind the first by
    the caller): the capture must not try to wait for the plan's own event of the warm-up calls."""
    import torch
    from paper_2503_18989_b200 import runner
    sc = _manual("fp16", 2, 128, [100, 900, 40], [300, 4, 64], 93)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    cur = torch.cuda.current_stream(cuda_device)
    for _ in range(2):
        ds.attend(stream=cur.cuda_stream)                      # earlier calls: the plan remembers this stream
    side = torch.cuda.Stream(device=cuda_device)
    side.wait_stream(cur)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        ds.attend(stream=side.cuda_stream)
    ds.out.fill_(float("nan")); ds.lse.fill_(float("nan"))
    graph.replay()
    go, gl = ds.results()
    _, _, want = oracle_replay(sc)
    assert_parity(go, want[0][0], "captured on another stream out")
    assert_parity(gl, want[0][1], "captured on another stream lse")
    ds.attend(stream=cur.cuda_stream)                          # and a plain call afterwards still works
    go, gl = ds.results()
    assert_parity(go, want[0][0], "plain call after the capture out")
    ds.close()


def test_calls_on_one_plan_from_two_streams_are_kept_in_order(cuda_device):
    """A plan serves one call at a time (its unit counter and status word are shared): calls handed different
    streams are ordered by the library itself, so alternating streams without any synchronisation is still correct."""
    import torch
    from paper_2503_18989_b200 import runner
    sc = W.ragged_prefill(num_requests=6, max_prefix=1024, H=4, seed=77)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    s1, s2 = torch.cuda.Stream(cuda_device), torch.cuda.Stream(cuda_device)
    torch.cuda.synchronize()
    for it in range(6):
        ds.attend(fused_append=True, stream=(s1 if it % 2 == 0 else s2).cuda_stream)
    out, lse = ds.results()
    _, _, want = oracle_replay(sc)
    assert_parity(out, want[0][0], "two streams out")
    assert_parity(lse, want[0][1], "two streams lse")
    ds.close()


def test_a_bf16_batch_with_wide_and_narrow_units_uses_both_tile_kernels(cuda_device):
    """bf16, head_dim 128: units of more than 128 rows run on CTA pairs and the narrower units of the same batch (a
    128-row remainder of a 384-row chunk, chunks of 128 / 64 / 17 rows) on single CTAs in a second grid with its own
    unit counter; every element against the oracle, twice in a row (the counters must be back at zero), also with key
    ranges cut and merged."""
    from paper_2503_18989_b200 import binding as B, runner
    prefix = [0, 300, 1000, 37, 2000, 640, 90, 5000]
    chunk = [512, 384, 128, 64, 300, 17, 4, 256]
    sc = _manual("bf16", 2, 128, prefix, chunk, 71)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.info["prefill_kernel"] == 3
    kp, vp, want = oracle_replay(sc)
    for _ in range(2):
        ds.out.fill_(float("nan")); ds.lse.fill_(float("nan"))
        ds.attend(fused_append=True)
        go, gl = ds.results()
        assert B.hat_last_device_status(ds.plan) == B.HAT_OK
        assert_parity(go, want[0][0], "wide + narrow out")
        assert_parity(gl, want[0][1], "wide + narrow lse")
    assert ds.canaries_intact()
    ds.close()


@pytest.mark.parametrize("seed,group,out16", [(1, 1, False), (2, 2, False), (3, 1, True)])
def test_random_bf16_batches_through_whatever_kernels_the_plan_picks(cuda_device, seed, group, out16):
    """Random bf16 batches (chunks of 1 .. 700 rows, prefixes of 0 .. 3000 tokens, some not page multiples; grouped query
    heads; 16-bit output): whichever mix of CTA-pair, one-CTA and streaming kernels and key-range cuts the plan picks,
    every element against the oracle."""
    import torch
    from paper_2503_18989_b200 import binding as B, runner
    rs = np.random.default_rng(100 + seed)
    R = 9
    chunk = [int(c) for c in rs.choice([1, 4, 16, 17, 64, 100, 128, 129, 200, 256, 300, 384, 512, 700], R)]
    prefix = [int(rs.integers(0, 3001)) for _ in range(R)]
    sc = _manual("bf16", 2, 128, prefix, chunk, 300 + seed, q_group=group)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    kp, vp, want = oracle_replay(sc)
    if out16:
        ds.attend16(fused_append=True)
        torch.cuda.synchronize()
        got = W.bits_to_f64(ds.out16.cpu().numpy().view(np.uint16), "bf16").reshape(want[0][0].shape)
        err = np.abs(got - want[0][0])
        assert np.all(err <= 2e-3 + np.abs(want[0][0]) * 2.0 ** -8), float(err.max())
    else:
        ds.attend(fused_append=True)
        go, gl = ds.results()
        assert_parity(go, want[0][0], f"random batch {seed} out")
        assert_parity(gl, want[0][1], f"random batch {seed} lse")
    assert B.hat_last_device_status(ds.plan) == B.HAT_OK
    assert ds.canaries_intact()
    gk, gv = cache.pools_to_host()
    assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
    ds.close()


# ----------------------------------------------------------------------------
# both tcgen05 tile kernels, whichever the plan would pick
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("kernel,code", [("pair", 3), ("tc5", 1)])
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_each_tcgen05_tile_kernel_on_every_kind_of_unit(cuda_device, kernel, code, dtype, monkeypatch):
    """Every element against the oracle with the tile kernel forced: full 256-row units, a 256 + 144 split, units of
    64 / 128 / 17 rows (half a CTA pair idles, results must not care), prefixes that are not page multiples, an empty
    prefix, grouped query heads, and streaming-class chunks in the same batch."""
    from paper_2503_18989_b200 import runner
    monkeypatch.setenv("HAT_PREFILL_KERNEL", kernel)
    prefix = [0, 1000, 77, 300, 2049, 5, 640, 33]
    chunk = [512, 400, 256, 64, 128, 17, 300, 4]
    sc = _manual(dtype, 2, 128, prefix, chunk, 81, q_group=2)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    assert ds.info["prefill_kernel"] == code
    ds.close()
    _check_full(sc, cuda_device)


@pytest.mark.parametrize("kernel", ["pair", "tc5"])
def test_each_tcgen05_tile_kernel_with_cut_key_ranges_and_sixteen_bit_output(cuda_device, kernel, monkeypatch):
    from paper_2503_18989_b200 import runner
    monkeypatch.setenv("HAT_PREFILL_KERNEL", kernel)
    monkeypatch.setenv("HAT_PREFILL_SPLIT_LEN", "384")          # key ranges of 384: partial rows, merge kernel, ragged last range
    sc = _manual("bf16", 3, 128, [900, 100, 1500], [512, 256, 300], 83)
    _check_full(sc, cuda_device)
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, cuda_device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    ds.attend(fused_append=True)
    out, lse = ds.results()
    ds.attend16(fused_append=False)
    import torch
    torch.cuda.synchronize()
    got = W.bits_to_f64(ds.out16.cpu().numpy().view(np.uint16), "bf16").reshape(out.shape)
    assert ds.canaries_intact()
    # the 16-bit rows are the fp32 rows rounded once: within half a unit in the last place (2^-8 relative) of them
    assert np.all(np.abs(got - out) <= np.abs(out) * 2.0 ** -8 + 1e-30)
