"""Writes tests/golden/tiny_rows.txt: out[:4] and lse of sampled (step, row, head) triples of the `tiny`
workload, computed by the CPU oracle only (never by the CUDA path).  The paper prints no worked
attention example, so these values pin the oracle + input recipe against silent drift; the oracle itself
is pinned to closed forms and invariants in tests/test_oracle_pins.py.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

from oracle import hat_oracle as O  # noqa: E402
from paper_2503_18989_b200 import workloads as W  # noqa: E402


def rows():
    sc = W.tiny()
    kp, vp = sc.k_pool.copy(), sc.v_pool.copy()
    rng = np.random.default_rng(2503_18989)
    out = []
    for s, st in enumerate(sc.steps):
        O.kv_append(sc.cache, kp, vp, st)
        o, l = O.chunk_attention(sc.cache, kp, vp, st)
        n = int(st.chunk_len[0])
        picks = sorted({0, n - 1, *[int(x) for x in rng.integers(0, n, size=3)]})
        for i in picks:
            h = int(rng.integers(sc.cache.num_heads))
            out.append((s, i, h, *[float(x) for x in o[i, h, :4]], float(l[i, h])))
    return out


if __name__ == "__main__":
    path = os.path.join(HERE, "tiny_rows.txt")
    with open(path, "w") as f:
        f.write("# tiny workload (1 request, 8 heads x 64, fp16, prompt 256 as 4 chunks of 64 + 4 draft tokens)\n")
        f.write("# written by tests/golden/make_golden.py from the CPU oracle; columns: step row head out0 out1 out2 out3 lse\n")
        for r in rows():
            f.write("%d %d %d %.17g %.17g %.17g %.17g %.17g\n" % r)
    print(path)
