"""The allocation-free entry point against the regular one.

Serving loops that run under CUDA-graph capture, or inside a framework that owns the whole device
heap, cannot call cudaMalloc, so they can create neither a plan nor a workspace.  For them the library
offers hat_verify_attention_static, whose split-KV partial results live in a fixed array inside the
library's device code.  This test drives it through the C ABI twice in a row on a draft-verification
batch (the second call reuses the scratch array the first one filled, with a different batch in
between) and compares out/lse with what hat_chunk_attention produces for the same inputs and with the CPU oracle.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

from paper_2503_18989_b200 import workloads as W

from common import ABS_TOL, REL_FLOOR, REL_TOL, assert_parity, oracle_replay

pytestmark = pytest.mark.gpu


def _regular(sc, device):
    """out/lse of the plan-based entry point, and the cache it left behind (chunk K/V appended)."""
    from paper_2503_18989_b200 import runner
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, device)
    ds = runner.DeviceStep(cache, sc.steps[0])
    ds.attend(fused_append=True)
    out, lse = ds.results()
    return cache, ds, out, lse


def _static(cache, ds, sc, device):
    import torch
    from paper_2503_18989_b200 import binding as B
    st = sc.steps[0]
    dev_i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
    cu, pl, cl, bt = dev_i32(st.cu_chunk), dev_i32(st.prefix_len), dev_i32(st.chunk_len), dev_i32(st.block_table)
    out = torch.full_like(ds.out, float("nan"))
    lse = torch.full_like(ds.lse, float("nan"))
    B.hat_verify_attention_static(cache.desc, st.num_requests, sc.cache.num_heads, int(st.chunk_len.max()),
                                  st.max_pages, cu, pl, cl, bt, ds.q, out, lse)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()


def _close(got, want, what):
    assert np.isfinite(got).all(), what
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    assert err.max() <= ABS_TOL, f"{what}: max-abs {err.max():.3e}"
    rel = (err / np.maximum(np.abs(want), REL_FLOOR)).max()
    assert rel <= REL_TOL, f"{what}: max-rel {rel:.3e}"


def test_static_entry_point_matches_regular_twice_in_a_row(cuda_device):
    first = W.spec_verify(num_requests=12, min_prefix=40, max_prefix=2500, max_draft=8, H=8, seed=901)
    other = W.spec_verify(num_requests=5, min_prefix=1, max_prefix=300, max_draft=16, H=4, d=64, dtype="bf16", seed=902)
    cache1, ds1, want_out1, want_lse1 = _regular(first, cuda_device)
    cache2, ds2, want_out2, want_lse2 = _regular(other, cuda_device)
    # call 1, a different batch (other geometry, so the scratch array is overwritten differently), call 1 again
    oracle = {id(sc): oracle_replay(sc)[2][0] for sc in (first, other)}
    for sc, cache, ds, wo, wl in ((first, cache1, ds1, want_out1, want_lse1),
                                  (other, cache2, ds2, want_out2, want_lse2),
                                  (first, cache1, ds1, want_out1, want_lse1)):
        got_out, got_lse = _static(cache, ds, sc, cuda_device)
        _close(got_out, wo, f"{sc.name} out")
        _close(got_lse, wl, f"{sc.name} lse")
        ref_out, ref_lse = oracle[id(sc)]
        assert_parity(got_out, ref_out, f"{sc.name} out vs oracle")
        assert_parity(got_lse, ref_lse, f"{sc.name} lse vs oracle")


def test_static_entry_point_leaves_skipped_rows_untouched(cuda_device):
    """Requests with chunk_len 0, and rows at or beyond max_chunk_len, are not computed: their out/lse rows keep
    the sentinel they held, and every other row still matches the oracle."""
    import torch
    from paper_2503_18989_b200 import binding as B
    sc = W.spec_verify(num_requests=6, min_prefix=20, max_prefix=600, max_draft=8, H=4, seed=904)
    st = sc.steps[0]
    cache, ds, _, _ = _regular(sc, cuda_device)
    ref_out, ref_lse = oracle_replay(sc)[2][0]
    dev_i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(cuda_device)
    cu, pl, bt = dev_i32(st.cu_chunk), dev_i32(st.prefix_len), dev_i32(st.block_table)
    # (a) request 2 announces chunk_len 0 to this call; (b) max_chunk_len 3 cuts every longer chunk to its first rows
    for zeroed, max_rows in ((2, 16), (None, 3)):
        cl_host = st.chunk_len.copy()
        if zeroed is not None:
            cl_host[zeroed] = 0
        out = torch.full_like(ds.out, float("nan"))
        lse = torch.full_like(ds.lse, float("nan"))
        B.hat_verify_attention_static(cache.desc, st.num_requests, sc.cache.num_heads, max_rows, st.max_pages,
                                      cu, pl, dev_i32(cl_host), bt, ds.q, out, lse)
        torch.cuda.synchronize()
        out, lse = out.cpu().numpy(), lse.cpu().numpy()
        computed = np.zeros(st.total_rows, dtype=bool)
        for r in range(st.num_requests):
            a = int(st.cu_chunk[r])
            n = min(int(cl_host[r]), max_rows)
            # a chunk cut short sees prefix + its own first rows only, which is what the oracle's rows say too
            computed[a:a + n] = True
        assert computed.any() and not computed.all()
        assert np.isnan(out[~computed]).all() and np.isnan(lse[~computed]).all()
        assert_parity(out[computed], ref_out[computed], "computed rows out")
        assert_parity(lse[computed], ref_lse[computed], "computed rows lse")


def test_static_entry_point_rejects_oversized_batches(cuda_device):
    from paper_2503_18989_b200 import binding as B
    sc = W.spec_verify(num_requests=2, min_prefix=10, max_prefix=40, H=2, seed=903)
    cache, ds, _, _ = _regular(sc, cuda_device)
    st = sc.steps[0]
    args = (st.max_pages, ds.q, ds.q, ds.q, ds.q, ds.q, ds.out, ds.lse)
    with pytest.raises(B.HatError) as e:         # 4000 requests x 8 ranges x 16 rows x 2 heads x 129 floats > 32 MiB
        B.hat_verify_attention_static(cache.desc, 4000, 2, 16, *args)
    assert e.value.status == B.HAT_ERR_TOO_LARGE
    with pytest.raises(B.HatError) as e:
        B.hat_verify_attention_static(cache.desc, 2, 2, 17, *args)
    assert e.value.status == B.HAT_ERR_INVALID_ARG
