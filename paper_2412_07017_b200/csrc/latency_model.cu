// Latency model of asynchronous function calling (paper Section 6.3, Appendix A): closed forms of the
// three execution models for a set of independent calls, the longest-processing-time-first order, and
// the completion times of an arbitrary generation order.  Host arithmetic only; it connects the
// microseconds of a decoding step (the attention kernels' output) to the paper's end-to-end latencies,
// and its completion times are where the interrupts of a replayed trace arrive.
#include <algorithm>
#include <numeric>
#include <vector>

#include "asynclm.h"

static bool valid(const double* gen, const double* exe, int32_t n) {
    if (n < 0 || (n > 0 && (!gen || !exe))) return false;
    for (int32_t i = 0; i < n; ++i)
        if (!(gen[i] > 0.0) || !(exe[i] > 0.0)) return false;      // the paper takes both positive
    return true;
}

extern "C" int asynclm_latency_model(const double* gen, const double* exe, int32_t n, asynclm_latency* out,
                                     int32_t* lpt_order) {
    if (!out || !valid(gen, exe, n) || n == 0) return ASYNCLM_ERR_INVALID_ARG;
    double sum_g = 0.0, sum_e = 0.0, max_e = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        sum_g += gen[i];
        sum_e += exe[i];
        max_e = std::max(max_e, exe[i]);
    }
    std::vector<int32_t> order((size_t)n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return exe[a] > exe[b]; });
    // under the LPT order call i completes at G(f_1) + ... + G(f_i) + E(f_i); the latest one ends the task
    double t = 0.0, worst = 0.0;
    for (int32_t k = 0; k < n; ++k) {
        t += gen[order[(size_t)k]];
        worst = std::max(worst, t + exe[order[(size_t)k]]);
    }
    out->l_sync = sum_g + sum_e;
    out->l_sync_par = sum_g + max_e;
    out->l_async = worst;
    out->speedup_estimate = 1.0 + (sum_e / n) / (sum_g / n);
    if (lpt_order) std::copy(order.begin(), order.end(), lpt_order);
    return ASYNCLM_OK;
}

extern "C" int asynclm_async_latency_of_order(const double* gen, const double* exe, const int32_t* order, int32_t n,
                                              double* latency, double* completion) {
    if (!latency || !order || !valid(gen, exe, n) || n == 0) return ASYNCLM_ERR_INVALID_ARG;
    std::vector<char> seen((size_t)n, 0);
    for (int32_t k = 0; k < n; ++k) {
        if (order[k] < 0 || order[k] >= n || seen[(size_t)order[k]]) return ASYNCLM_ERR_INVALID_ARG;
        seen[(size_t)order[k]] = 1;
    }
    double t = 0.0, worst = 0.0;
    for (int32_t k = 0; k < n; ++k) {
        const int32_t i = order[k];
        t += gen[i];
        if (completion) completion[i] = t + exe[i];
        worst = std::max(worst, t + exe[i]);
    }
    *latency = worst;
    return ASYNCLM_OK;
}
