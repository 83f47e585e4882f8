"""The cloud-side controller (state monitor Eq. 1-2, chunk size Eq. 3, parallel-drafting steps Eq. 6):
closed forms pin the Python oracle, and the C ABI implementation is compared with the oracle on seeded
random histories.  Host code only."""
import math

import numpy as np
import pytest

from oracle.hat_ctrl_oracle import Ctrl as OracleCtrl
from paper_2503_18989_b200 import binding as B


def _both(alpha=0.8, w=64.0, n=256, hat_lib=None):
    return OracleCtrl(alpha, w, n), B.Ctrl(alpha, w, n, 8)


# ---------------------------------------------------------------- pins of the oracle
def test_moving_average_closed_form():
    a = 0.8
    o = OracleCtrl(a, 64.0, 256)
    obs = [100.0, 300.0, 50.0, 700.0, 700.0]
    for t, m in enumerate(obs, 1):
        o.observe(m, 1.0)
        want = a ** (t - 1) * obs[0] + (1 - a) * sum(a ** (t - k) * obs[k - 1] for k in range(2, t + 1))
        assert o.mu == pytest.approx(want, rel=1e-14)
    o = OracleCtrl(0.0, 64.0, 256)          # alpha = 0: no memory
    o.observe(10, 1); o.observe(640, 2)
    assert o.mu == 640 and o.predict(640) == 2
    o = OracleCtrl(1.0, 64.0, 256)          # alpha = 1: frozen at the first observation
    o.observe(128, 3); o.observe(6400, 9)
    assert o.mu == 128 and o.predict(128) == 3


def test_device_moving_average_closed_form():
    # Sec. 3.2: the per-device drafting delay and link bandwidths are averaged with the same weight as Eq. 1.
    # Two DIFFERENT observations: new = alpha * old + (1 - alpha) * x2, for each of the three quantities.
    a = 0.8
    o = OracleCtrl(a, 64.0, 256)
    x1, x2, x3 = (0.010, 6e6, 11e6), (0.030, 9e6, 14e6), (0.020, 5e6, 12e6)
    o.device_observe(2, *x1)
    assert o.dev[2] == list(x1)                                  # the first observation is taken as it is
    o.device_observe(2, *x2)
    for got, u, v in zip(o.dev[2], x1, x2):
        assert got == pytest.approx(a * u + (1 - a) * v, rel=1e-15)
    assert o.dev[2][0] == pytest.approx(0.014, rel=1e-12)         # 0.8 * 10 ms + 0.2 * 30 ms, by hand
    assert o.dev[2][1] == pytest.approx(6.6e6, rel=1e-12)
    assert o.dev[2][2] == pytest.approx(11.6e6, rel=1e-12)
    o.device_observe(2, *x3)
    for got, u, v, w in zip(o.dev[2], x1, x2, x3):
        assert got == pytest.approx(a * a * u + a * (1 - a) * v + (1 - a) * w, rel=1e-15)
    assert 5 not in o.dev                                         # other devices untouched
    o = OracleCtrl(0.0, 64.0, 256)                                # alpha = 0: the latest observation
    o.device_observe(0, *x1); o.device_observe(0, *x2)
    assert o.dev[0] == list(x2)
    o = OracleCtrl(1.0, 64.0, 256)                                # alpha = 1: frozen at the first
    o.device_observe(0, *x1); o.device_observe(0, *x2)
    assert o.dev[0] == list(x1)


def test_linear_delay_is_reproduced_and_extrapolated():
    # two observed grid points of g(x) = 2e-3 + 1e-5 x (alpha = 0: mu^t = mu_hat^t) define the whole line
    ga, gb = 2e-3, 1e-5
    o = OracleCtrl(0.0, 64.0, 256)
    for x in (256.0, 1024.0):
        o.observe(x, ga + gb * x)
    for x in (0.0, 100.0, 256.0, 700.0, 1024.0, 5000.0):
        assert o.predict(x) == pytest.approx(ga + gb * x, rel=1e-12)


def test_chunk_size_closed_forms():
    A, P = 8192.0, 4                     # fp16 hidden state of 4096, pipeline length 4
    beta = 7.5e6                         # 7.5 MB/s upload
    # constant g: X * A / beta = 2 g / P  =>  X = 2 g beta / (A P)
    o = OracleCtrl(0.8, 64.0, 256)
    o.observe(512.0, 0.050)
    o.device_observe(0, 0.02, beta, 12e6)
    assert o.chunk_size(0, A, P, 1, 4096) == math.ceil(2 * 0.050 * beta / (A * P))
    # linear g = a + b x:  X A / beta = (2 a + 2 b mu + b X) / P  =>  X (A P / beta - b) = 2 a + 2 b mu
    ga, gb = 0.020, 4e-5
    o = OracleCtrl(0.0, 64.0, 256)
    o.observe(1024.0, ga + gb * 1024.0); o.observe(256.0, ga + gb * 256.0)      # mu ends at 256
    o.device_observe(0, 0.02, beta, 12e6)
    root = (2 * ga + 2 * gb * 256.0) / (A * P / beta - gb)
    assert o.chunk_size(0, A, P, 1, 4096) == math.ceil(root - 1e-9)
    assert 13.9 < root < 14.0
    assert o.chunk_size(0, A, P, 1, 10) == 10                                    # clamped from above
    assert o.chunk_size(0, A, P, 500, 4096) == 500                               # clamped from below


def test_parallel_draft_steps_by_hand():
    o = OracleCtrl(0.8, 64.0, 256)
    o.observe(320.0, 0.030)
    o.device_observe(3, 0.012, 8e6, 16e6)
    # 4 draft tokens of 8192 bytes: 4.096 ms up + 30 ms in the cloud + 2.048 ms down = 36.144 ms; / 12 ms = 3.01
    assert o.parallel_draft_steps(3, 4, 8192.0) == 3
    o.device_observe(3, 0.012, 8e6, 16e6)
    assert o.parallel_draft_steps(3, 0, 8192.0) == 2                             # 30 ms / 12 ms


# ---------------------------------------------------------------- the C ABI against the oracle
@pytest.mark.parametrize("seed", range(6))
def test_library_matches_oracle_on_random_histories(hat_lib, seed):
    rng = np.random.default_rng(seed)
    alpha = [0.8, 0.5, 0.0, 1.0, 0.9, 0.3][seed]
    o, c = _both(alpha, 64.0, 128)
    for dev in range(3):
        for _ in range(int(rng.integers(1, 4))):
            args = (float(rng.uniform(0.005, 0.05)), float(rng.uniform(5e6, 10e6)), float(rng.uniform(10e6, 15e6)))
            o.device_observe(dev, *args); B.hat_ctrl_device_observe(c, dev, *args)
        assert B.hat_ctrl_device_state(c, dev) == pytest.approx(tuple(o.dev[dev]), rel=1e-14)
    for t in range(60):
        mu_hat = float(rng.integers(1, 6000))
        eta_hat = 0.004 + 2e-5 * mu_hat * float(rng.uniform(0.8, 1.2))           # roughly linear delay, noisy
        o.observe(mu_hat, eta_hat); B.hat_ctrl_observe(c, mu_hat, eta_hat)
        assert B.hat_ctrl_mu(c) == pytest.approx(o.mu, rel=1e-14)
        for x in (0.0, 37.0, o.mu, o.mu + 512.0, 9000.0):
            assert B.hat_ctrl_predict(c, x) == pytest.approx(o.predict(x), rel=1e-12, abs=1e-15)
        dev = int(rng.integers(3))
        A, P = [8192.0, 10240.0][t % 2], [1, 2, 4, 8][t % 4]
        assert B.hat_ctrl_chunk_size(c, dev, A, P, 16, 2048) == o.chunk_size(dev, A, P, 16, 2048)
        n = int(rng.integers(0, 9))
        assert B.hat_ctrl_parallel_draft_steps(c, dev, n, A) == o.parallel_draft_steps(dev, n, A)


def test_controller_argument_errors(hat_lib):
    import ctypes as C
    h = C.c_void_p()
    assert hat_lib.hat_ctrl_create(1.5, 64.0, 16, 4, C.byref(h)) == B.HAT_ERR_INVALID_ARG
    assert hat_lib.hat_ctrl_create(0.8, 0.0, 16, 4, C.byref(h)) == B.HAT_ERR_INVALID_ARG
    c = B.Ctrl(0.8, 64.0, 16, 2)
    with pytest.raises(B.HatError):
        B.hat_ctrl_chunk_size(c, 0, 8192.0, 4, 1, 100)          # device never observed
    with pytest.raises(B.HatError):
        B.hat_ctrl_device_observe(c, 5, 0.01, 1e6, 1e6)         # device out of range
    with pytest.raises(B.HatError):
        B.hat_ctrl_observe(c, -1.0, 0.1)
    assert B.hat_ctrl_predict(c, 100.0) == 0.0                  # nothing observed yet
    assert hat_lib.hat_ctrl_destroy(None) == B.HAT_OK
