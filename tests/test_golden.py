"""Stored oracle values for the tiny workload (tests/golden/tiny_rows.txt, written by make_golden.py from the
oracle alone): the oracle must still reproduce them, and the CUDA path must match them within tolerance."""
import os

import numpy as np
import pytest

from paper_2503_18989_b200 import workloads as W

from common import ABS_TOL, oracle_replay

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_rows.txt")


def _load():
    rows = [ln.split() for ln in open(GOLDEN) if not ln.startswith("#")]
    return [(int(r[0]), int(r[1]), int(r[2]), np.array([float(x) for x in r[3:7]]), float(r[7])) for r in rows]


def test_oracle_reproduces_stored_values():
    _, _, res = oracle_replay(W.tiny())
    rows = _load()
    assert len(rows) >= 15
    for s, i, h, out4, lse in rows:
        assert np.allclose(res[s][0][i, h, :4], out4, rtol=0, atol=1e-12)    # libm may differ in the last bit
        assert abs(res[s][1][i, h] - lse) <= 1e-12


@pytest.mark.gpu
def test_cuda_path_matches_stored_values(cuda_device):
    from paper_2503_18989_b200 import runner
    _, got = runner.run_scenario(W.tiny(), cuda_device)
    for s, i, h, out4, lse in _load():
        assert np.max(np.abs(got[s][0][i, h, :4] - out4)) <= ABS_TOL
        assert abs(got[s][1][i, h] - lse) <= ABS_TOL
