// Optimal speculation stride scheduler (OS^3): host-side arithmetic only.
// Section 4 ("Optimal speculation stride scheduler") defines the objective, Appendix A.2 the
// expected number of verified documents and the estimator of the speculation accuracy.
#include <cmath>

#include "../../include/ralm.h"

extern "C" {

double ralm_os3_expected_verified(double gamma, int32_t s) {
    if (s <= 0) return 0.0;
    if (gamma <= 0.0) return 1.0;
    if (gamma >= 1.0) return static_cast<double>(s);
    return (1.0 - std::pow(gamma, s)) / (1.0 - gamma);
}

double ralm_os3_objective(double gamma, double a, double b, int32_t s, int32_t async_verify) {
    if (s <= 0) return 0.0;
    const double verified = ralm_os3_expected_verified(gamma, s);
    const double sync_latency = s * a + b;
    double latency = sync_latency;
    if (async_verify) {
        const double all_match = gamma <= 0.0 ? 0.0 : (gamma >= 1.0 ? 1.0 : std::pow(gamma, s));
        const double overlapped = (s - 1) * a + (a > b ? a : b);
        latency = all_match * overlapped + (1.0 - all_match) * sync_latency;
    }
    return latency > 0.0 ? verified / latency : INFINITY;
}

ralm_status_t ralm_os3_gamma(const int32_t *matched, const int32_t *strides, int32_t w, double gamma_max,
                             double *gamma_out) {
    if (!gamma_out || w < 0 || (w > 0 && (!matched || !strides)) || !(gamma_max >= 0.0)) return RALM_ERR_INVALID_ARG;
    long long hits = 0, misses = 0;
    for (int32_t t = 0; t < w; ++t) {
        if (strides[t] < 1 || matched[t] < 0 || matched[t] > strides[t]) return RALM_ERR_INVALID_ARG;
        hits += matched[t];
        misses += matched[t] < strides[t] ? 1 : 0;
    }
    double g = (hits + misses) > 0 ? static_cast<double>(hits) / static_cast<double>(hits + misses) : 0.0;
    if (g > gamma_max) g = gamma_max;
    *gamma_out = g;
    return RALM_OK;
}

ralm_status_t ralm_os3_stride(const int32_t *matched, const int32_t *strides, int32_t w, double gamma_max,
                              double a, double b, int32_t s_max, int32_t async_verify, int32_t *s_out) {
    if (!s_out || s_max < 1 || !(a >= 0.0) || !(b >= 0.0)) return RALM_ERR_INVALID_ARG;
    double gamma = 0.0;
    const ralm_status_t rs = ralm_os3_gamma(matched, strides, w, gamma_max, &gamma);
    if (rs != RALM_OK) return rs;
    int32_t best_s = 1;
    double best = ralm_os3_objective(gamma, a, b, 1, async_verify);
    for (int32_t s = 2; s <= s_max; ++s) {
        const double v = ralm_os3_objective(gamma, a, b, s, async_verify);
        if (v > best) {  // ties keep the shorter stride
            best = v;
            best_s = s;
        }
    }
    *s_out = best_s;
    return RALM_OK;
}

}  // extern "C"
