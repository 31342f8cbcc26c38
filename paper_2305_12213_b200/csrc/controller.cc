// Host-side proportional batch-size controller (Section 3.3, Eq. 4-5).
//
// Compiled without FMA contraction: the integer batch sizes must come out the
// same on every host, so each fp64 operation below is a separately rounded
// IEEE operation in the order written.
#include <cmath>
#include <cstdint>
#include <vector>

#include "dynbatch.h"

namespace {

struct Bounds {
    const int32_t* lo;
    const int32_t* hi;
    int64_t total;
    int64_t lower(int k) const { return lo ? lo[k] : 1; }
    int64_t upper(int k) const { return hi ? hi[k] : total; }
};

// Real targets -> integers within the bounds that sum to `total`: floor, then
// move single units to/from the worker whose integer is furthest from its
// target on the needed side; the first such worker wins a tie.
db_status to_integers(const std::vector<double>& target, const Bounds& bd,
                      std::vector<int64_t>& out) {
    const int K = static_cast<int>(target.size());
    int64_t min_sum = 0, max_sum = 0;
    for (int k = 0; k < K; ++k) {
        if (bd.lower(k) < 0 || bd.upper(k) < bd.lower(k)) return DB_ERR_ARG;
        min_sum += bd.lower(k);
        max_sum += bd.upper(k);
    }
    if (min_sum > bd.total || max_sum < bd.total) return DB_ERR_INFEASIBLE;

    out.resize(K);
    int64_t have = 0;
    for (int k = 0; k < K; ++k) {
        const double fl = std::floor(target[k]);
        int64_t x;
        if (fl > static_cast<double>(bd.total)) x = bd.total;
        else if (fl < 0.0) x = 0;
        else x = static_cast<int64_t>(fl);
        if (x < bd.lower(k)) x = bd.lower(k);
        if (x > bd.upper(k)) x = bd.upper(k);
        out[k] = x;
        have += x;
    }
    for (; have < bd.total; ++have) {
        int pick = -1;
        double deficit = 0.0;
        for (int k = 0; k < K; ++k) {
            if (out[k] >= bd.upper(k)) continue;
            const double d = target[k] - static_cast<double>(out[k]);
            if (pick < 0 || d > deficit) { pick = k; deficit = d; }
        }
        ++out[pick];
    }
    for (; have > bd.total; --have) {
        int pick = -1;
        double excess = 0.0;
        for (int k = 0; k < K; ++k) {
            if (out[k] <= bd.lower(k)) continue;
            const double d = static_cast<double>(out[k]) - target[k];
            if (pick < 0 || d > excess) { pick = k; excess = d; }
        }
        --out[pick];
    }
    return DB_OK;
}

}  // namespace

extern "C" db_status db_controller_step_ex(int32_t* b, const double* throughputs,
                                           int32_t K, double kp,
                                           const int32_t* b_min,
                                           const int32_t* b_max) {
    if (!b || !throughputs) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K) return DB_ERR_ARG;
    if (!(kp > 0.0) || !(kp <= 1.0)) return DB_ERR_ARG;
    int64_t total = 0;
    for (int k = 0; k < K; ++k) {
        if (b[k] < 0) return DB_ERR_ARG;
        if (!std::isfinite(throughputs[k]) || !(throughputs[k] > 0.0)) return DB_ERR_ARG;
        total += b[k];
    }
    if (total <= 0 || total > INT32_MAX) return DB_ERR_ARG;

    // iteration times implied by the throughputs, and their mean
    std::vector<double> t(K);
    double t_sum = 0.0;
    for (int k = 0; k < K; ++k) {
        t[k] = static_cast<double>(b[k]) / throughputs[k];
        t_sum += t[k];
    }
    const double t_bar = t_sum / static_cast<double>(K);

    // Eq. 4-5 with gain kp, then rescale to the global batch
    std::vector<double> target(K);
    double moved_sum = 0.0;
    for (int k = 0; k < K; ++k) {
        const double tau = t[k] - t_bar;
        const double delta = -throughputs[k] * tau;
        target[k] = static_cast<double>(b[k]) + kp * delta;
        moved_sum += target[k];
    }
    for (int k = 0; k < K; ++k)
        target[k] = target[k] * static_cast<double>(total) / moved_sum;

    std::vector<int64_t> next;
    const db_status st = to_integers(target, Bounds{b_min, b_max, total}, next);
    if (st != DB_OK) return st;
    for (int k = 0; k < K; ++k) b[k] = static_cast<int32_t>(next[k]);
    return DB_OK;
}

extern "C" db_status db_controller_step(int32_t* b, const double* throughputs,
                                        int32_t K, double kp) {
    return db_controller_step_ex(b, throughputs, K, kp, nullptr, nullptr);
}
