// Cloud-side control plane of HAT (host code only): the state monitor's moving averages (Sec. 3.2, Eq. 1-2), the
// chunk-size rule of the prompt-chunking module (Sec. 3.3, Eq. 3) and the number of parallel-drafting steps
// (Sec. 3.5, Eq. 6).  The delay predictor g(.) is fed with the measured delay of the attention step of this library
// (or of a whole middle-submodel step) per batched token size.
//
// Readings where the paper is silent: g is kept on a uniform grid of token sizes; an observation updates, by Eq. 2,
// the grid point nearest to the smoothed batched token size; between observed grid points g is linear, beyond the
// outermost two it continues with their slope (Sec. 2.3 reports a near-linear delay beyond 512 tokens), and with a
// single observed point it is constant.  A grid point observed for the first time takes the observation itself
// (there is no g^{t-1} to average with); the same holds for the first observation of every moving average.
#include <cmath>
#include <new>
#include <vector>

#include "../../include/hat.h"

struct hat_ctrl {
    double alpha;
    double bin_width;
    bool has_mu;
    double mu;                         // Eq. 1
    std::vector<double> g;             // Eq. 2, one value per grid point
    std::vector<unsigned char> seen;
    struct Device { bool seen; double gamma, beta_up, beta_down; };
    std::vector<Device> dev;
};

namespace {

// g(x) from the observed grid points (see the header comment for the interpolation rule).
double predict(const hat_ctrl* c, double x) {
    const int n = (int)c->g.size();
    int first = -1, last = -1;
    for (int i = 0; i < n; ++i)
        if (c->seen[i]) { if (first < 0) first = i; last = i; }
    if (first < 0) return 0.0;
    if (first == last) return c->g[first];
    const double pos = x / c->bin_width;
    // neighbours among the observed points
    int lo = -1, hi = -1;
    for (int i = 0; i < n; ++i) {
        if (!c->seen[i]) continue;
        if ((double)i <= pos) lo = i;
        if ((double)i >= pos && hi < 0) hi = i;
    }
    if (lo < 0) {                       // left of every observation: slope of the first two
        lo = first;
        for (hi = first + 1; !c->seen[hi]; ++hi) { }
    } else if (hi < 0) {                // right of every observation: slope of the last two
        hi = last;
        for (lo = last - 1; !c->seen[lo]; --lo) { }
    } else if (lo == hi) {
        return c->g[lo];
    }
    const double t = (pos - lo) / (double)(hi - lo);
    const double v = c->g[lo] + t * (c->g[hi] - c->g[lo]);
    return v > 0.0 ? v : 0.0;
}

}  // namespace

extern "C" {

int hat_ctrl_create(double alpha, double bin_width, int num_bins, int max_devices, hat_ctrl** out) {
    if (!out) return HAT_ERR_INVALID_ARG;
    *out = nullptr;
    if (!(alpha >= 0.0 && alpha <= 1.0) || !(bin_width > 0.0) || num_bins < 2 || num_bins > (1 << 20) || max_devices < 0 ||
        max_devices > (1 << 20))
        return HAT_ERR_INVALID_ARG;
    hat_ctrl* c = new (std::nothrow) hat_ctrl();
    if (!c) return HAT_ERR_INVALID_ARG;
    c->alpha = alpha;
    c->bin_width = bin_width;
    c->has_mu = false;
    c->mu = 0.0;
    c->g.assign(num_bins, 0.0);
    c->seen.assign(num_bins, 0);
    c->dev.assign(max_devices, hat_ctrl::Device{false, 0.0, 0.0, 0.0});
    *out = c;
    return HAT_OK;
}

int hat_ctrl_destroy(hat_ctrl* c) {
    delete c;
    return HAT_OK;
}

int hat_ctrl_observe(hat_ctrl* c, double mu_hat, double eta_hat) {
    if (!c || !(mu_hat >= 0.0) || !(eta_hat >= 0.0) || !std::isfinite(mu_hat) || !std::isfinite(eta_hat)) return HAT_ERR_INVALID_ARG;
    // Eq. 1
    c->mu = c->has_mu ? c->alpha * c->mu + (1.0 - c->alpha) * mu_hat : mu_hat;
    c->has_mu = true;
    // Eq. 2 at the grid point nearest to mu^t
    long i = std::lround(c->mu / c->bin_width);
    if (i < 0) i = 0;
    if (i >= (long)c->g.size()) i = (long)c->g.size() - 1;
    c->g[i] = c->seen[i] ? c->alpha * c->g[i] + (1.0 - c->alpha) * eta_hat : eta_hat;
    c->seen[i] = 1;
    return HAT_OK;
}

int hat_ctrl_mu(const hat_ctrl* c, double* out) {
    if (!c || !out) return HAT_ERR_INVALID_ARG;
    *out = c->mu;
    return HAT_OK;
}

int hat_ctrl_predict(const hat_ctrl* c, double tokens, double* out) {
    if (!c || !out || !std::isfinite(tokens)) return HAT_ERR_INVALID_ARG;
    *out = predict(c, tokens);
    return HAT_OK;
}

int hat_ctrl_device_observe(hat_ctrl* c, int device, double gamma_hat, double beta_up_hat, double beta_down_hat) {
    if (!c || device < 0 || device >= (int)c->dev.size()) return HAT_ERR_INVALID_ARG;
    if (!(gamma_hat > 0.0) || !(beta_up_hat > 0.0) || !(beta_down_hat > 0.0)) return HAT_ERR_INVALID_ARG;
    hat_ctrl::Device& d = c->dev[device];
    const double a = c->alpha;
    if (d.seen) {
        d.gamma = a * d.gamma + (1.0 - a) * gamma_hat;
        d.beta_up = a * d.beta_up + (1.0 - a) * beta_up_hat;
        d.beta_down = a * d.beta_down + (1.0 - a) * beta_down_hat;
    } else {
        d = hat_ctrl::Device{true, gamma_hat, beta_up_hat, beta_down_hat};
    }
    return HAT_OK;
}

int hat_ctrl_device_state(const hat_ctrl* c, int device, double* gamma, double* beta_up, double* beta_down) {
    if (!c || device < 0 || device >= (int)c->dev.size() || !c->dev[device].seen) return HAT_ERR_INVALID_ARG;
    if (gamma) *gamma = c->dev[device].gamma;
    if (beta_up) *beta_up = c->dev[device].beta_up;
    if (beta_down) *beta_down = c->dev[device].beta_down;
    return HAT_OK;
}

int hat_ctrl_chunk_size(const hat_ctrl* c, int device, double bytes_per_token, int pipeline_length, int x_min, int x_max,
                        int* out) {
    if (!c || !out || device < 0 || device >= (int)c->dev.size() || !c->dev[device].seen) return HAT_ERR_INVALID_ARG;
    if (!(bytes_per_token > 0.0) || pipeline_length < 1 || x_min < 1 || x_max < x_min) return HAT_ERR_INVALID_ARG;
    const double beta = c->dev[device].beta_up;
    const double g_mu = predict(c, c->mu);
    // Eq. 3: upload time of the chunk = (waiting + computing) / P.  f is negative at 0 and, while uploading a token
    // costs more than it adds to the predicted delay, increasing: the smallest integer with f >= 0 is found by bisection.
    auto f = [&](double x) { return x * bytes_per_token / beta - (g_mu + predict(c, c->mu + x)) / pipeline_length; };
    if (f((double)x_min) >= 0.0) { *out = x_min; return HAT_OK; }
    if (f((double)x_max) < 0.0) { *out = x_max; return HAT_OK; }
    int lo = x_min, hi = x_max;          // f(lo) < 0 <= f(hi)
    while (hi - lo > 1) {
        const int mid = lo + (hi - lo) / 2;
        if (f((double)mid) >= 0.0) hi = mid; else lo = mid;
    }
    *out = hi;
    return HAT_OK;
}

int hat_ctrl_parallel_draft_steps(const hat_ctrl* c, int device, int draft_len, double bytes_per_token, int* out) {
    if (!c || !out || device < 0 || device >= (int)c->dev.size() || !c->dev[device].seen) return HAT_ERR_INVALID_ARG;
    if (draft_len < 0 || !(bytes_per_token > 0.0)) return HAT_ERR_INVALID_ARG;
    const hat_ctrl::Device& d = c->dev[device];
    // Eq. 6: what fits, at gamma per drafting step, into upload + in-cloud delay + download of the draft sequence
    const double window = draft_len * bytes_per_token / d.beta_up + predict(c, c->mu) + draft_len * bytes_per_token / d.beta_down;
    const double steps = std::floor(window / d.gamma);
    *out = steps > 2147483647.0 ? 2147483647 : (int)steps;
    return HAT_OK;
}

}  // extern "C"
