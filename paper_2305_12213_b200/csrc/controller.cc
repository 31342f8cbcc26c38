// Host-side proportional batch-size controller (Section 3.3, Eq. 4-5).
//
// Compiled without FMA contraction: the integer batch sizes must come out the
// same on every host, so each fp64 operation below is a separately rounded
// IEEE operation in the order written.
#include <cmath>
#include <cstdint>
#include <new>
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

// ---------------------------------------------------------------------------
// Slice of the parameters owned by one of several parameter servers (Section 4)
// ---------------------------------------------------------------------------
extern "C" db_status db_shard_range(int64_t N, int32_t G, int32_t r, int32_t align, int64_t* begin, int64_t* end) {
    if (!begin || !end) return DB_ERR_NULL;
    if (N < 0 || G < 1 || r < 0 || r >= G || align < 1) return DB_ERR_ARG;
    int64_t chunk = (N + G - 1) / G;
    chunk = (chunk + align - 1) / align * align;
    const int64_t lo = static_cast<int64_t>(r) * chunk, hi = lo + chunk;
    *begin = lo < N ? lo : N;
    *end = hi < N ? hi : N;
    return DB_OK;
}

// ---------------------------------------------------------------------------
// Static open-loop allocation (Section 3.2)
// ---------------------------------------------------------------------------
extern "C" db_status db_static_allocate(const double* throughputs, int32_t K, int32_t b0,
                                        const int32_t* b_min, const int32_t* b_max, int32_t* b) {
    if (!throughputs || !b) return DB_ERR_NULL;
    if (K < 1 || K > DB_MAX_K || b0 < 1) return DB_ERR_ARG;
    double x_sum = 0.0;
    for (int k = 0; k < K; ++k) {
        if (!std::isfinite(throughputs[k]) || !(throughputs[k] > 0.0)) return DB_ERR_ARG;
        x_sum += throughputs[k];
    }
    const int64_t total = static_cast<int64_t>(K) * b0;
    if (total > INT32_MAX) return DB_ERR_ARG;
    std::vector<double> target(K);
    for (int k = 0; k < K; ++k) target[k] = static_cast<double>(total) * throughputs[k] / x_sum;
    std::vector<int64_t> out;
    const db_status st = to_integers(target, Bounds{b_min, b_max, total}, out);
    if (st != DB_OK) return st;
    for (int k = 0; k < K; ++k) b[k] = static_cast<int32_t>(out[k]);
    return DB_OK;
}

// ---------------------------------------------------------------------------
// Stabilised controller (Section 3.3.1): EWMA, bounds (optionally learnt), dead-band
// ---------------------------------------------------------------------------
struct db_controller {
    int K = 0;
    double kp = 1.0, alpha = 0.5, dead_band = 0.05;
    bool adaptive = false, has_min = false, has_max = false;
    std::vector<int32_t> b, b_min, b_max, prev_b, learnt_max;
    std::vector<double> ewma, prev_x;
    int samples_since_readjust = 0;
};

extern "C" db_status db_controller_create(db_controller** out, const int32_t* b0, int32_t K, double kp,
                                          double alpha, double dead_band, const int32_t* b_min,
                                          const int32_t* b_max, int32_t adaptive_b_max) {
    if (!out || !b0) return DB_ERR_NULL;
    *out = nullptr;
    if (K < 1 || K > DB_MAX_K) return DB_ERR_ARG;
    if (!(kp > 0.0) || !(kp <= 1.0) || !(alpha > 0.0) || !(alpha <= 1.0) || !(dead_band >= 0.0)) return DB_ERR_ARG;
    for (int k = 0; k < K; ++k) {
        if (b0[k] < 1) return DB_ERR_ARG;
        // A worker at b = 0 has no iteration time to observe, so the handle's lower bounds start at 1.
        if (b_min && b_min[k] < 1) return DB_ERR_ARG;
        if (b_max && b_max[k] < (b_min ? b_min[k] : 1)) return DB_ERR_ARG;
    }
    db_controller* c = new (std::nothrow) db_controller();
    if (!c) return DB_ERR_ARG;
    c->K = K;
    c->kp = kp;
    c->alpha = alpha;
    c->dead_band = dead_band;
    c->adaptive = adaptive_b_max != 0;
    c->b.assign(b0, b0 + K);
    c->has_min = b_min != nullptr;
    c->has_max = b_max != nullptr;
    if (b_min) c->b_min.assign(b_min, b_min + K);
    if (b_max) c->b_max.assign(b_max, b_max + K);
    c->prev_b.assign(K, 0);
    c->learnt_max.assign(K, 0);
    c->ewma.assign(K, 0.0);
    c->prev_x.assign(K, 0.0);
    *out = c;
    return DB_OK;
}

extern "C" db_status db_controller_destroy(db_controller* c) {
    delete c;
    return DB_OK;
}

extern "C" db_status db_controller_observe(db_controller* c, const double* iteration_times, int32_t* b_out,
                                           int32_t* changed) {
    if (!c || !iteration_times) return DB_ERR_NULL;
    const int K = c->K;
    for (int k = 0; k < K; ++k)
        if (!std::isfinite(iteration_times[k]) || !(iteration_times[k] > 0.0)) return DB_ERR_ARG;

    // 1. smoothed iteration times since the last readjustment
    for (int k = 0; k < K; ++k)
        c->ewma[k] = c->samples_since_readjust == 0
                         ? iteration_times[k]
                         : c->alpha * iteration_times[k] + (1.0 - c->alpha) * c->ewma[k];
    c->samples_since_readjust += 1;

    // 2. throughput seen by the proportional rule
    std::vector<double> x(K);
    int64_t total = 0;
    for (int k = 0; k < K; ++k) {
        x[k] = static_cast<double>(c->b[k]) / c->ewma[k];
        total += c->b[k];
    }

    // 3. bounds; an upper bound is learnt when raising a worker's batch lowered its throughput
    const int32_t* lo = c->has_min ? c->b_min.data() : nullptr;
    const int32_t* hi_user = c->has_max ? c->b_max.data() : nullptr;
    std::vector<int32_t> hi(K);
    bool use_learnt = false;
    if (c->adaptive) {
        for (int k = 0; k < K; ++k)
            if (c->prev_x[k] > 0.0 && c->b[k] > c->prev_b[k] && x[k] < c->prev_x[k])
                if (c->learnt_max[k] == 0 || c->prev_b[k] < c->learnt_max[k]) c->learnt_max[k] = c->prev_b[k];
        for (int k = 0; k < K; ++k) {
            int64_t h = hi_user ? hi_user[k] : total;
            if (c->learnt_max[k] > 0 && c->learnt_max[k] < h) {
                h = c->learnt_max[k];
                use_learnt = true;
            }
            hi[k] = static_cast<int32_t>(h);
        }
    }
    std::vector<int32_t> next(c->b);
    db_status st = DB_ERR_INFEASIBLE;
    if (use_learnt) st = db_controller_step_ex(next.data(), x.data(), K, c->kp, lo, hi.data());
    if (st == DB_ERR_INFEASIBLE) {
        next = c->b;
        st = db_controller_step_ex(next.data(), x.data(), K, c->kp, lo, hi_user);
    }
    if (changed) *changed = 0;
    if (st != DB_OK) return st;

    // 4. dead-band on the integer result: all workers move, or none
    double worst = 0.0;
    for (int k = 0; k < K; ++k) {
        const double rel = std::fabs(static_cast<double>(next[k]) - static_cast<double>(c->b[k])) /
                           static_cast<double>(c->b[k]);
        if (rel > worst) worst = rel;
    }
    if (worst > c->dead_band) {
        if (c->adaptive)
            for (int k = 0; k < K; ++k) {
                c->prev_b[k] = c->b[k];
                c->prev_x[k] = x[k];
            }
        c->b = next;
        c->samples_since_readjust = 0;
        if (changed) *changed = 1;
    }
    if (b_out)
        for (int k = 0; k < K; ++k) b_out[k] = c->b[k];
    return DB_OK;
}
