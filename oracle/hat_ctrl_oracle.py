"""Plain-Python oracle of HAT's cloud-side control laws (TEST INFRASTRUCTURE ONLY).

State monitor: moving averages of the batched token size mu and of the predictive delay function g (Sec. 3.2,
Eq. 1 and Eq. 2, alpha in [0, 1]); chunk size X_i from  X_i * A / beta_up = (g(mu) + g(mu + X_i)) / P  (Sec. 3.3,
Eq. 3); parallel-drafting steps lambda_i = floor((mu_i A / beta_up + g(mu) + mu_i A / beta_down) / gamma_i)
(Sec. 3.5, Eq. 6).  Written from the equations, in their notation; it shares no code with the library.

Readings where the paper is silent (the library documents the same ones): g lives on a uniform grid of token sizes;
Eq. 2 updates the grid point nearest to mu^t; g is linear between observed points, keeps the outermost slope beyond
them, is constant with one observed point and 0 with none; the first observation of a moving average is taken as it
is; Eq. 3 is answered with the smallest integer X in [x_min, x_max] whose upload time reaches the right-hand side.

Pins (tests/test_ctrl.py): the closed form of an exponential moving average (of mu, and of the per-device
quantities with two different observations), exact reproduction of a linear g,
the closed-form root of Eq. 3 for constant and for linear g, Eq. 6 evaluated by hand.
"""
import math


class Ctrl:
    def __init__(self, alpha=0.8, bin_width=64.0, num_bins=256):
        self.alpha, self.w, self.n = alpha, bin_width, num_bins
        self.mu = None
        self.g = {}                      # grid index -> g value (observed points only)
        self.dev = {}                    # device -> [gamma, beta_up, beta_down]

    # Eq. 1 and Eq. 2
    def observe(self, mu_hat, eta_hat):
        a = self.alpha
        self.mu = mu_hat if self.mu is None else a * self.mu + (1 - a) * mu_hat
        i = min(max(int(math.floor(self.mu / self.w + 0.5)), 0), self.n - 1)
        self.g[i] = eta_hat if i not in self.g else a * self.g[i] + (1 - a) * eta_hat

    def device_observe(self, i, gamma, beta_up, beta_down):
        a = self.alpha
        new = [gamma, beta_up, beta_down]
        self.dev[i] = new if i not in self.dev else [a * o + (1 - a) * v for o, v in zip(self.dev[i], new)]

    def predict(self, x):
        pts = sorted(self.g)
        if not pts:
            return 0.0
        if len(pts) == 1:
            return self.g[pts[0]]
        pos = x / self.w
        below = [i for i in pts if i <= pos]
        above = [i for i in pts if i >= pos]
        if not below:
            lo, hi = pts[0], pts[1]
        elif not above:
            lo, hi = pts[-2], pts[-1]
        else:
            lo, hi = below[-1], above[0]
            if lo == hi:
                return self.g[lo]
        v = self.g[lo] + (pos - lo) / (hi - lo) * (self.g[hi] - self.g[lo])
        return max(v, 0.0)

    # Eq. 3, by exhaustive search (the definition: smallest integer that satisfies the inequality)
    def chunk_size(self, i, A, P, x_min, x_max):
        beta = self.dev[i][1]
        g_mu = self.predict(self.mu)
        for X in range(x_min, x_max + 1):
            if X * A / beta >= (g_mu + self.predict(self.mu + X)) / P:
                return X
        return x_max

    # Eq. 6
    def parallel_draft_steps(self, i, mu_i, A):
        gamma, up, down = self.dev[i]
        return int(math.floor((mu_i * A / up + self.predict(self.mu) + mu_i * A / down) / gamma))
