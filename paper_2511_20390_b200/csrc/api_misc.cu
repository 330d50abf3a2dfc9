// Error strings and other small host-only entry points.
#include "common.cuh"
#include <vector>

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
