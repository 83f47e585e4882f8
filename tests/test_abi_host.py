"""Host-side tests of the C-ABI library: it loads, exports what include/hat.h declares, rejects bad
arguments before any launch, and schedules batches sensibly.  No test here needs a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2503_18989_b200 import binding as B
from paper_2503_18989_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "hat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hat_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(hat_lib):
    declared = _declared_symbols()
    assert "hat_kv_append" in declared and "hat_chunk_attention" in declared
    for name in declared:
        assert hasattr(hat_lib, name), f"{name} is declared in hat.h but not exported"
    assert sorted(B.EXPORTS) == declared, "binding and header disagree on the entry points"


def test_version_and_status_strings(hat_lib):
    assert B.hat_version() == 110
    seen = {B.hat_status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert B.hat_status_string(-99) == "unknown status"


def _cache(dtype="fp16", num_pages=64, H=4, d=128, **over):
    spec = W.CacheSpec(dtype, H, d, num_pages, "paged")
    kw = dict(dtype=dtype, num_pages=num_pages, num_kv_heads=H, head_dim=d, stride_page=spec.stride_page,
              stride_token=spec.stride_token, stride_head=spec.stride_head)
    kw.update(over)
    return B.make_cache_desc(**kw)


def _plan(cache, prefix, chunk, table, H=4, cu=None, flags=B.HAT_PLAN_HOST_ONLY):
    prefix = np.asarray(prefix, np.int32)
    chunk = np.asarray(chunk, np.int32)
    if cu is None:
        cu = np.concatenate([[0], np.cumsum(chunk)]).astype(np.int32)
    return B.hat_plan_create(cache, H, cu, prefix, chunk, np.asarray(table, np.int32), flags)


def _status(fn, *a, **k):
    try:
        fn(*a, **k)
    except B.HatError as e:
        return e.status
    return B.HAT_OK


def test_plan_rejects_bad_arguments(hat_lib):
    c = _cache()
    ok_table = [[0, 1, 2, 3]]
    assert _status(_plan, c, [10], [20], ok_table) == B.HAT_OK
    # cu_chunk not the prefix sum of chunk_len
    assert _status(_plan, c, [10], [20], ok_table, cu=np.array([0, 19], np.int32)) == B.HAT_ERR_INVALID_ARG
    assert _status(_plan, c, [10], [20], ok_table, cu=np.array([1, 21], np.int32)) == B.HAT_ERR_INVALID_ARG
    assert _status(_plan, c, [-1], [20], ok_table) == B.HAT_ERR_INVALID_ARG
    assert _status(_plan, c, [10], [-2], ok_table, cu=np.array([0, -2], np.int32)) == B.HAT_ERR_INVALID_ARG
    # table too short / page outside the pool / unused entries may be anything
    assert _status(_plan, c, [60], [20], ok_table) == B.HAT_ERR_OUT_OF_RANGE
    assert _status(_plan, c, [10], [20], [[0, 64, 2, 3]]) == B.HAT_ERR_OUT_OF_RANGE
    assert _status(_plan, c, [10], [20], [[0, -1, 2, 3]]) == B.HAT_ERR_OUT_OF_RANGE
    assert _status(_plan, c, [10], [20], [[0, 1, -1, 9999]]) == B.HAT_OK
    # a page written by two requests; reading a shared page is fine
    assert _status(_plan, c, [0, 0], [5, 5], [[7], [7]]) == B.HAT_ERR_OUT_OF_RANGE
    assert _status(_plan, c, [16, 16], [5, 5], [[7, 8], [7, 9]]) == B.HAT_OK
    # unsupported geometry
    assert _status(_plan, _cache(page_size=32), [0], [4], [[0]]) == B.HAT_ERR_UNSUPPORTED
    assert _status(_plan, _cache(head_dim=96), [0], [4], [[0]]) == B.HAT_ERR_UNSUPPORTED
    assert _status(_plan, _cache(dtype=2), [0], [4], [[0]]) == B.HAT_ERR_UNSUPPORTED
    assert _status(_plan, _cache(stride_token=132), [0], [4], [[0]]) == B.HAT_ERR_UNSUPPORTED
    assert _status(_plan, c, [0], [4], [[0]], H=8) == B.HAT_OK                    # two query heads per K/V head
    assert _status(_plan, c, [0], [4], [[0]], H=6) == B.HAT_ERR_UNSUPPORTED       # not a multiple of the K/V heads
    assert _status(_plan, c, [0], [4], [[0]], H=2) == B.HAT_ERR_UNSUPPORTED
    # null descriptors
    out = C.c_void_p()
    assert hat_lib.hat_plan_create(None, None, C.byref(out)) == B.HAT_ERR_INVALID_ARG
    assert hat_lib.hat_plan_create(C.byref(c), None, None) == B.HAT_ERR_INVALID_ARG
    assert hat_lib.hat_plan_destroy(None) == B.HAT_OK


def test_empty_batches_are_valid(hat_lib):
    c = _cache()
    p = _plan(c, [], [], np.zeros((0, 0), np.int32))
    assert B.hat_plan_get_info(p).total_rows == 0
    p = _plan(c, [5, 0], [0, 0], [[0], [1]])
    info = B.hat_plan_get_info(p).as_dict()
    assert info["total_rows"] == 0 and info["num_verify_items"] == 0 and info["workspace_bytes"] == 0


def test_host_only_plan_cannot_launch(hat_lib):
    c = _cache()
    p = _plan(c, [10], [4], [[0]])
    assert hat_lib.hat_kv_append(C.byref(c), p.handle, None, None, None) == B.HAT_ERR_INVALID_ARG
    assert hat_lib.hat_qkv_rope_append(C.byref(c), p.handle, None, 64, None, None, C.c_float(10000.0), 0,
                                       None) == B.HAT_ERR_INVALID_ARG
    assert hat_lib.hat_qkv_rope_append(None, None, None, 64, None, None, C.c_float(10000.0), 0, None) == B.HAT_ERR_INVALID_ARG


def _info(sc, step=0, **env):
    st = sc.steps[step]
    spec = sc.cache
    c = B.make_cache_desc(spec.dtype, spec.num_pages, spec.num_heads, spec.head_dim, spec.stride_page,
                          spec.stride_token, spec.stride_head)
    p = B.hat_plan_create(c, spec.num_heads, st.cu_chunk, st.prefix_len, st.chunk_len, st.block_table,
                          B.HAT_PLAN_HOST_ONLY)
    return B.hat_plan_get_info(p).as_dict()


def _shapes_only(maker, **kw):
    """Scenario with 1 head x 64 so that building it is cheap; shapes are what matters here."""
    return maker(H=1, d=64, **kw)


def test_schedule_of_the_verify_batch(hat_lib):
    sc = _shapes_only(W.spec_verify)
    st = sc.steps[0]
    info = _info(sc)
    assert info["num_verify_requests"] == 30 and info["num_prefill_requests"] == 0
    assert info["max_splits"] <= 32
    L = info["verify_split_len"]
    assert L % 16 == 0 and L >= 16
    def pieces(n):                       # ranges of L keys, lengthened so that no request has more than 32
        per = max(L, -(-(-(-n // 32)) // 16) * 16)
        return -(-n // per)
    want_items = sum(pieces(int(p + c)) for p, c in zip(st.prefix_len, st.chunk_len))
    assert info["num_verify_items"] == want_items
    split_rows = sum(int(c) for p, c in zip(st.prefix_len, st.chunk_len) if pieces(int(p + c)) > 1)
    assert info["num_merge_rows"] == split_rows
    # flops and bytes follow the stated conventions
    d, H = 64, 1
    F = sum(4 * d * H * (int(c) * int(p) + int(c) * (int(c) + 1) // 2) for p, c in zip(st.prefix_len, st.chunk_len))
    Bk = sum(2 * (int(p) + int(c)) * H * d * 2 for p, c in zip(st.prefix_len, st.chunk_len))
    assert info["attn_flops"] == F and info["kv_read_bytes"] == Bk


def test_schedule_of_prefill_and_mixed_batches(hat_lib):
    sc = _shapes_only(W.ragged_prefill)
    st = sc.steps[0]
    info = _info(sc)
    assert info["num_prefill_requests"] == 30 and info["num_verify_requests"] == 0
    rows = info["prefill_tile_rows"]
    tiles = sum(-(-int(c) // rows) for c in st.chunk_len)
    assert info["num_prefill_items"] >= tiles
    sc = _shapes_only(W.mixed_13b)
    info = _info(sc)
    assert info["num_prefill_requests"] == 8 and info["num_verify_requests"] == 32
    assert info["total_rows"] == 8 * 512 + 32 * 4
    assert info["max_splits"] <= 32


def test_small_prefill_batches_are_cut_to_fill_one_round_of_the_persistent_kernel(hat_lib):
    """One request of 256 rows x 32 heads is 32 units for 148 persistent CTAs.  The plan cuts its keys into ranges
    chosen by a cost model (a step, the fixed cost of a unit, the merge pass): the ranges are multiples of 128 keys,
    no more than one unit per CTA results, and a short request is left whole because cutting it costs more than it
    saves."""
    c = _cache(num_pages=256, H=32)
    table = [list(range(144))]
    sms = 148                                                  # what a host-only plan assumes
    for prefix in (1024, 1792):
        info = B.hat_plan_get_info(_plan(c, [prefix], [256], table, H=32)).as_dict()
        L = info["prefill_split_len"]
        assert info["prefill_kernel"] == 1 and L >= 256 and L % 128 == 0
        assert info["max_splits"] == -(-(prefix + 256) // L) and info["max_splits"] > 1
        assert sms // 2 < info["num_prefill_items"] * 32 <= sms
        assert info["num_merge_rows"] == 256
    info = B.hat_plan_get_info(_plan(c, [0], [256], table, H=32)).as_dict()
    assert info["prefill_split_len"] == 0 and info["num_merge_rows"] == 0 and info["workspace_bytes"] == 0


def test_grouped_query_heads_change_the_work_but_not_the_cache_traffic(hat_lib):
    c = _cache(num_pages=64, H=4, d=128)
    table = [list(range(40))]
    one = B.hat_plan_get_info(_plan(c, [600], [4], table, H=4)).as_dict()
    four = B.hat_plan_get_info(_plan(c, [600], [4], table, H=16)).as_dict()
    assert four["attn_flops"] == 4 * one["attn_flops"] and four["kv_read_bytes"] == one["kv_read_bytes"]
    assert four["num_verify_requests"] == 1 and four["total_rows"] == 4


def test_long_request_never_exceeds_32_key_ranges(hat_lib):
    c = _cache(num_pages=4096)
    n = 60000
    table = [list(range((n + 4 + 15) // 16))]
    p = _plan(c, [n], [4], table)
    info = B.hat_plan_get_info(p).as_dict()
    assert info["max_splits"] <= 32 and info["num_verify_items"] == info["max_splits"]


def test_batches_beyond_the_launch_limits_are_rejected(hat_lib):
    # 70000 one-token requests = 70000 streaming work items: more than one grid dimension can index
    n = 70000
    c = _cache(num_pages=n, H=1, d=64)
    table = np.arange(n, dtype=np.int32)[:, None]
    assert _status(_plan, c, np.zeros(n, np.int32), np.ones(n, np.int32), table, H=1) == B.HAT_ERR_TOO_LARGE
    assert _status(_plan, c, np.zeros(60000, np.int32), np.ones(60000, np.int32), table[:60000], H=1) == B.HAT_OK


def test_static_entry_point_clamps_unvalidated_lengths(hat_lib):
    """hat_verify_attention_static reads its lengths from device memory nobody checked; the helper that turns them
    into key ranges must keep every block-table lookup inside the request's row whatever they hold."""
    S = B.HAT_STATIC_SPLITS
    # a sane request: the ranges tile [0, P + C) in whole pages, in order
    ranges = [B.hat_static_key_range(1000, 5, 8, 100, sp) for sp in range(S)]
    assert all(r[0] == 1000 and r[1] == 5 for r in ranges)
    assert ranges[0][2] == 0 and ranges[-1][3] == 1005
    for a, b in zip(ranges, ranges[1:]):
        assert a[3] == b[2] and a[2] % 16 == 0 and a[2] <= a[3]
    per = ((1005 + S - 1) // S + 15) // 16 * 16
    assert ranges[0][3] == per
    # overstated, negative and oversized lengths (nothing here is sent to a GPU)
    rng = np.random.default_rng(7)
    cases = [(10**9, 16, 16, 5), (-5, 3, 8, 4), (0, 10**6, 16, 1), (79, 16, 16, 5), (80, 1, 16, 5), (2**31 - 1, 2**31 - 1, 16, 3)]
    cases += [(int(rng.integers(-100, 5000)), int(rng.integers(-5, 40)), int(rng.integers(1, 17)), int(rng.integers(1, 64)))
              for _ in range(200)]
    for P, Cl, max_rows, max_pages in cases:
        cover = 0
        for sp in range(S):
            prefix, rows, b, e = B.hat_static_key_range(P, Cl, max_rows, max_pages, sp)
            assert 0 <= prefix and 0 <= rows <= max_rows and prefix + rows <= max_pages * 16
            assert 0 <= b <= e <= prefix + rows
            assert e == b or (e - 1) // 16 <= max_pages - 1          # last page looked up is a column of the table row
            assert b == cover
            cover = e
        assert cover == prefix + rows
        if 0 <= P and 0 <= Cl <= max_rows and P + Cl <= max_pages * 16:
            assert (prefix, rows) == (P, Cl)                          # valid lengths pass through unchanged
    with pytest.raises(B.HatError):
        B.hat_static_key_range(10, 2, 17, 4, 0)
    with pytest.raises(B.HatError):
        B.hat_static_key_range(10, 2, 8, 4, S)


def test_choice_of_the_tile_kernel(hat_lib):
    """The CTA-pair kernel takes the units of more than 128 rows: for bf16 in every batch that has some (narrower units
    of the same batch run on single CTAs), for fp16 only when every unit is that wide and long (2500 keys on average)
    and there are at least 1.5 of them per SM; head_dim 64 keeps the one-CTA tcgen05 kernel."""
    def info(prefix, chunk, H, d=128, dtype="bf16"):
        rng = np.random.Generator(np.random.PCG64(3))
        table, num_pages = W._place_pages(rng, np.asarray(prefix) + np.asarray(chunk), slack_pages=2)
        c = B.make_cache_desc(dtype, num_pages, H, d, H * 16 * d, d, 16 * d)
        cu = np.concatenate([[0], np.cumsum(chunk)]).astype(np.int32)
        p = B.hat_plan_create(c, H, cu, np.asarray(prefix, np.int32), np.asarray(chunk, np.int32), table,
                              B.HAT_PLAN_HOST_ONLY)
        return B.hat_plan_get_info(p).as_dict()
    assert info([100] * 8, [512] * 8, 40)["prefill_kernel"] == 3              # 16 wide units x 40 heads
    assert info([100] * 8 + [700] * 4, [512] * 8 + [4] * 4, 40)["prefill_kernel"] == 3   # short chunks do not matter
    assert info([100] * 8, [512] * 7 + [384], 40)["prefill_kernel"] == 3       # bf16: the 128-row unit of the 384 goes to a single CTA
    assert info([100] * 8, [512] * 7 + [400], 40)["prefill_kernel"] == 3       # 400 = 256 + 144: both halves in use
    assert info([100] * 8, [128] * 8, 40)["prefill_kernel"] == 1               # nothing for a pair
    assert info([100] * 8, [512] * 7 + [384], 40, dtype="fp16")["prefill_kernel"] == 1   # fp16: only batches of full units
    assert info([100] * 2, [512] * 2, 32)["prefill_kernel"] == 3               # bf16: small batches too
    assert info([100], [256], 8)["prefill_kernel"] == 3
    assert info([100] * 2, [512] * 2, 32, dtype="fp16")["prefill_kernel"] == 1   # fp16: 4 x 32 = 128 units < 222
    assert info([4000] * 3, [512] * 3, 40, dtype="fp16")["prefill_kernel"] == 3   # 6 x 40 = 240 long units
    assert info([4000] * 8, [512] * 8, 40, dtype="fp16")["prefill_kernel"] == 3
    assert info([1000] * 8, [512] * 8, 40, dtype="fp16")["prefill_kernel"] == 1    # fp16 units of ~1400 keys: no gain on pairs
    assert info([100] * 8, [4] * 8, 40)["prefill_kernel"] == 1                 # no tile-class chunk at all
    assert info([100] * 8, [512] * 8, 40, d=64)["prefill_kernel"] == 1
