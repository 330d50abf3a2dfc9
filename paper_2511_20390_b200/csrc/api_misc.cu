// Error strings and other small host-only entry points.
#include "common.cuh"
#include <vector>
#include <cmath>

#include <atomic>
static std::atomic<int> g_launch_overlap{1};
bool free_launch_overlap_enabled() { return g_launch_overlap.load(std::memory_order_relaxed) != 0; }
extern "C" int free_set_launch_overlap(int on) { return g_launch_overlap.exchange(on ? 1 : 0); }

extern "C" const char* free_strerror(int code) {
    switch (code) {
        case FREE_OK: return "ok";
        case FREE_ERR_ARG: return "invalid argument (null pointer, negative count or bad enum)";
        case FREE_ERR_SHAPE: return "inconsistent or out-of-range dimensions";
        case FREE_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case FREE_ERR_UNSUPPORTED: return "configuration not supported by the kernels";
        case FREE_ERR_SIGMA: return "variance not positive and finite";
        case FREE_ERR_WORKSPACE: return "workspace missing or too small";
        case FREE_ERR_CUDA: return "CUDA call failed";
        case FREE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error code";
    }
}

// Relaxation profile from measured prediction deviations (Sec. 3.4): a non-decreasing fit (weighted pool-adjacent-
// violators), a centred moving average that keeps it non-decreasing, then lambda_n = g_first / g_n.
extern "C" int free_fit_lambda_profile(const double* eps_delta, const int64_t* count, int N, int window, float* lambda_out) {
    if (!eps_delta || !lambda_out) return FREE_ERR_ARG;
    if (N < 1 || window < 0) return FREE_ERR_SHAPE;
    // transitions without a measurement take the nearest measured value (the earlier one on a tie)
    std::vector<double> y(N), wt(N, 1.0);
    std::vector<int> valid;
    for (int n = 0; n < N; ++n) {
        const bool ok = (!count || count[n] > 0) && eps_delta[n] == eps_delta[n] && eps_delta[n] >= 0.0;
        if (ok) valid.push_back(n);
    }
    if (valid.empty()) return FREE_ERR_SHAPE;
    size_t vi = 0;
    for (int n = 0; n < N; ++n) {
        while (vi + 1 < valid.size() && abs(valid[vi + 1] - n) < abs(valid[vi] - n)) ++vi;
        y[n] = eps_delta[valid[vi]];
        wt[n] = (count && count[n] > 0 && valid[vi] == n) ? (double)count[n] : 1.0;
    }
    // pool adjacent violators: blocks of (weighted mean, weight, length)
    std::vector<double> bm, bw; std::vector<int> bl;
    for (int n = 0; n < N; ++n) {
        bm.push_back(y[n]); bw.push_back(wt[n]); bl.push_back(1);
        while (bm.size() > 1 && bm[bm.size() - 2] > bm.back()) {
            const size_t k = bm.size() - 1;
            const double w2 = bw[k - 1] + bw[k];
            bm[k - 1] = (bm[k - 1] * bw[k - 1] + bm[k] * bw[k]) / w2;
            bw[k - 1] = w2; bl[k - 1] += bl[k];
            bm.pop_back(); bw.pop_back(); bl.pop_back();
        }
    }
    std::vector<double> g; g.reserve(N);
    for (size_t k = 0; k < bm.size(); ++k) for (int i = 0; i < bl[k]; ++i) g.push_back(bm[k]);
    // centred moving average over 2*window+1 points, the ends held
    std::vector<double> sm(N);
    for (int n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int o = -window; o <= window; ++o) { int i = n + o; i = i < 0 ? 0 : (i >= N ? N - 1 : i); acc += g[i]; }
        sm[n] = acc / (2 * window + 1);
    }
    for (int n = 0; n < N; ++n) lambda_out[n] = sm[n] > 0.0 ? (float)(sm[0] / sm[n] > 1.0 ? 1.0 : sm[0] / sm[n]) : 1.0f;
    return FREE_OK;
}

// Reverse-process tables from a list of betas (Eq. ddpm_update, Sec. 4's posterior variance, Appendix "Variance
// Setting", Eq. mean_var_gamma).  fp64 throughout; abar is the running product in index order.
static int schedule_tables(const std::vector<double>& beta, int variance_mode, double variance_weight, double stochasticity,
                           double* coef_x, double* coef_eps, double* sigma2) {
    if (variance_mode != FREE_VAR_POSTERIOR && variance_mode != FREE_VAR_BETA && variance_mode != FREE_VAR_INTERP) return FREE_ERR_ARG;
    if (stochasticity < 0.0 && variance_mode == FREE_VAR_INTERP && !(variance_weight >= 0.0 && variance_weight <= 1.0)) return FREE_ERR_SHAPE;
    const int N = (int)beta.size();
    double abar = 1.0;
    for (int s = 0; s < N; ++s) {
        const double b = beta[s];
        if (!(b > 0.0 && b < 1.0)) return FREE_ERR_SHAPE;
        const double alpha = 1.0 - b, abar_prev = abar;
        abar *= alpha;
        if (stochasticity >= 0.0) {
            const double e2 = stochasticity * stochasticity;
            coef_x[s] = 1.0 + 0.5 * b;
            coef_eps[s] = 0.5 * (1.0 + e2) * b / std::sqrt(1.0 - abar);
            sigma2[s] = e2 * b;
        } else {
            coef_x[s] = 1.0 / std::sqrt(alpha);
            coef_eps[s] = b / (std::sqrt(1.0 - abar) * std::sqrt(alpha));
            const double post = b * (1.0 - abar_prev) / (1.0 - abar);
            sigma2[s] = variance_mode == FREE_VAR_POSTERIOR ? post
                      : variance_mode == FREE_VAR_BETA ? b
                      : (s == 0 ? 0.0 : std::pow(b, variance_weight) * std::pow(post, 1.0 - variance_weight));
        }
    }
    sigma2[0] = 0.0;
    return FREE_OK;
}

// beta_s on a line from first to last, both ends exact
static std::vector<double> linear_betas(int n, double first, double last) {
    std::vector<double> b(n);
    const double step = (last - first) / (double)(n - 1);
    for (int s = 0; s < n; ++s) b[s] = first + (double)s * step;
    b[n - 1] = last;
    return b;
}

extern "C" int free_schedule_linear(int N, double beta_first, double beta_last, int variance_mode, double variance_weight,
                                    double stochasticity, double* coef_x, double* coef_eps, double* sigma2, double* t_embed_value) {
    if (!coef_x || !coef_eps || !sigma2 || !t_embed_value) return FREE_ERR_ARG;
    if (N < 2) return FREE_ERR_SHAPE;
    const int rc = schedule_tables(linear_betas(N, beta_first, beta_last), variance_mode, variance_weight, stochasticity, coef_x, coef_eps, sigma2);
    if (rc != FREE_OK) return rc;
    for (int s = 0; s < N; ++s) t_embed_value[s] = (double)s;
    return FREE_OK;
}

extern "C" int free_schedule_respaced(int N, int n_full, double beta_first, double beta_last, int variance_mode, double variance_weight,
                                      double stochasticity, double* coef_x, double* coef_eps, double* sigma2, double* t_embed_value) {
    if (!coef_x || !coef_eps || !sigma2 || !t_embed_value) return FREE_ERR_ARG;
    if (N < 2 || n_full < N) return FREE_ERR_SHAPE;
    const std::vector<double> full = linear_betas(n_full, beta_first, beta_last);
    std::vector<double> abar_full(n_full);
    double run = 1.0;
    for (int s = 0; s < n_full; ++s) {
        if (!(full[s] > 0.0 && full[s] < 1.0)) return FREE_ERR_SHAPE;
        run *= 1.0 - full[s];
        abar_full[s] = run;
    }
    std::vector<double> beta(N);
    double prev = 1.0;
    for (int i = 0; i < N; ++i) {
        const long keep = std::lrint((double)i * ((double)(n_full - 1) / (double)(N - 1)));   // round half to even (default mode)
        t_embed_value[i] = (double)keep;
        beta[i] = 1.0 - abar_full[keep] / prev;
        prev = abar_full[keep];
    }
    return schedule_tables(beta, variance_mode, variance_weight, stochasticity, coef_x, coef_eps, sigma2);
}
