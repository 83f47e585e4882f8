"""Shared helpers of the tests: oracle replay of a scenario and the parity criterion."""
import numpy as np

from oracle import hat_oracle as O

ABS_TOL = 2e-3     # max-abs error bound (fp16/bf16 inputs, fp32 accumulation)
REL_TOL = 1e-2     # max-rel error bound, measured against max(|ref|, REL_FLOOR)
REL_FLOOR = 0.1


def oracle_replay(sc):
    """Run every step of a scenario through the oracle: append, then attend.
    Returns (k_pool, v_pool, [(out, lse) per step]) as numpy arrays."""
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    res = []
    for st in sc.steps:
        O.kv_append(sc.cache, kp, vp, st)
        res.append(O.chunk_attention(sc.cache, kp, vp, st))
    return kp, vp, res


def parity_errors(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    if got.size == 0:
        return 0.0, 0.0
    err = np.abs(got - ref)
    rel = err / np.maximum(np.abs(ref), REL_FLOOR)
    return float(np.nanmax(err)) if not np.isnan(err).any() else float("nan"), \
        float(np.nanmax(rel)) if not np.isnan(rel).any() else float("nan")


def assert_parity(got, ref, what=""):
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the GPU result"
    max_abs, max_rel = parity_errors(got, ref)
    assert max_abs <= ABS_TOL, f"{what}: max-abs {max_abs:.3e} > {ABS_TOL}"
    assert max_rel <= REL_TOL, f"{what}: max-rel {max_rel:.3e} > {REL_TOL}"
    return max_abs, max_rel
