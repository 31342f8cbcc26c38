/*
 * ref_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of the parameter-server step of
 * dynamic-batching BSP training (Tyagi & Sharma, "Taming Resource
 * Heterogeneity In Distributed ML Training With Dynamic Batching"):
 *
 *   - batch-proportional gradient weights            (Section 3.1, Eq. 2)
 *   - weighted aggregate + parameter update          (Section 3.1, Eq. 3)
 *     with the heavy-ball momentum optimizer the paper trains ResNet-50
 *     with (Section 4, workloads paragraph)
 *   - the proportional batch-size controller         (Section 3.3, Eq. 4-5)
 *     and its stabilised form                        (Section 3.3.1)
 *   - the static throughput-proportional allocation  (Section 3.2)
 *   - the mean cross-entropy gradient of a bias-free linear-softmax
 *     classifier, used to check the weighting against the gradient of the
 *     concatenated batch (Section 3.1: the weights sum to one, so equal
 *     batches give the plain mean of Eq. 1).
 *
 * Only tests, the smoke check and the CPU-baseline timing may call this
 * file.  It shares no code, header or table with the CUDA library and is
 * never a fallback for it.  Everything is written as the definition reads:
 * one loop per sum, k ascending, no blocking or fusion.  The OpenMP pragma
 * on the element loop only spreads independent elements j over host cores
 * for the timed baseline; every element's arithmetic is untouched by it.
 *
 * Parity pins (tests/test_oracle_pins.py): equal batches reduce to the plain
 * mean (Eq. 1); K = 1 is the identity; scaling every b by a constant changes
 * nothing; the aggregate of per-worker softmax gradients equals the gradient
 * of the concatenated batch (brute force); heavy-ball closed form for a
 * constant gradient and the torch.optim.SGD trajectory; finite differences of
 * the loss; controller fixed point, one-step closed form b*tbar/t (Section
 * 3.3), sum conservation, exhaustive check of the integer apportionment;
 * for the stabilised controller pandas' EWMA, the dead-band at 0.05 and three
 * traces worked by hand (learnt bounds that cannot hold the global batch, a
 * bound learnt twice, the smoothed comparison at every observation), the
 * dead-band's exact form (largest relative move, against the batch in use,
 * strictly above the threshold) and the return of surplus units.
 * tests/test_oracle_mutations.py plants single errors in a copy of this file
 * and requires the pins to fail for each.
 * Nothing here is left "parity unpinned".
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define REF_OK 0
#define REF_ERR_ARG 2
#define REF_ERR_INFEASIBLE 4

#define REF_F32 0
#define REF_BF16 1

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
static double widen_bf16(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double grad_at(const void* g, int dtype, int64_t j) {
    if (dtype == REF_BF16) return widen_bf16(((const uint16_t*)g)[j]);
    return (double)((const float*)g)[j];
}

/* Eq. 2: lambda_k = b_k / sum_i b_i, so that sum_k lambda_k = 1. */
int ref_weights(const int32_t* b, int32_t K, double* lambda) {
    if (!b || !lambda || K < 1) return REF_ERR_ARG;
    int64_t S = 0;
    for (int32_t k = 0; k < K; ++k) {
        if (b[k] < 0) return REF_ERR_ARG;
        S += b[k];
    }
    if (S <= 0) return REF_ERR_ARG;
    for (int32_t k = 0; k < K; ++k) lambda[k] = (double)b[k] / (double)S;
    return REF_OK;
}

/*
 * Eq. 2-3 with heavy-ball momentum.  grads[k] is worker k's MEAN gradient
 * over its b_k samples (N stored values, fp32 or bf16).  For each element j:
 *     g   = sum_k lambda_k * g_k[j]          (k ascending; b_k = 0 is skipped
 *                                             and its buffer is never read)
 *     v_j = mu * v_j + g
 *     p_j = p_j - lr * v_j
 * Reading of Eq. 3: the printed extra 1/K in front of the step is not
 * applied -- with sum lambda = 1 it would break the stated equivalence with
 * Eq. 1; a caller wanting it passes lr/K.  State p, v is fp64 in and out
 * (callers widen stored fp32 exactly); g_out (nullable) receives g;
 * sq_out (nullable) receives sum_j g^2.
 */
int ref_aggregate_update(const void* const* grads, int32_t grad_dtype,
                         const int32_t* b, int32_t K, int64_t N,
                         double* p, double* v, double lr, double mu,
                         double* g_out, double* sq_out) {
    if (!grads || !b || K < 1 || N < 0) return REF_ERR_ARG;
    if (grad_dtype != REF_F32 && grad_dtype != REF_BF16) return REF_ERR_ARG;
    if (N > 0 && (!p || !v)) return REF_ERR_ARG;
    double* lambda = (double*)malloc(sizeof(double) * (size_t)K);
    if (!lambda) return REF_ERR_ARG;
    int rc = ref_weights(b, K, lambda);
    if (rc != REF_OK) { free(lambda); return rc; }
    double sq = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : sq)
    for (int64_t j = 0; j < N; ++j) {
        double g = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            if (b[k] == 0) continue;
            g += lambda[k] * grad_at(grads[k], grad_dtype, j);
        }
        v[j] = mu * v[j] + g;
        p[j] = p[j] - lr * v[j];
        if (g_out) g_out[j] = g;
        sq += g * g;
    }
    if (sq_out) *sq_out = sq;
    free(lambda);
    return REF_OK;
}

/*
 * The same weighted aggregate followed by Adam, the optimizer of the paper's
 * MNIST workload (Section 4).  The paper prints no formula; this is the
 * textbook rule (Kingma & Ba, Algorithm 1) with bias correction at step t>=1:
 *     m = b1*m + (1-b1)*g;  u = b2*u + (1-b2)*g^2
 *     p = p - lr * (m/(1-b1^t)) / (sqrt(u/(1-b2^t)) + eps)
 */
int ref_aggregate_adam(const void* const* grads, int32_t grad_dtype,
                       const int32_t* b, int32_t K, int64_t N,
                       double* p, double* m, double* u, double lr,
                       double beta1, double beta2, double eps, int64_t t,
                       double* g_out, double* sq_out) {
    if (!grads || !b || K < 1 || N < 0 || t < 1) return REF_ERR_ARG;
    if (grad_dtype != REF_F32 && grad_dtype != REF_BF16) return REF_ERR_ARG;
    if (N > 0 && (!p || !m || !u)) return REF_ERR_ARG;
    double* lambda = (double*)malloc(sizeof(double) * (size_t)K);
    if (!lambda) return REF_ERR_ARG;
    int rc = ref_weights(b, K, lambda);
    if (rc != REF_OK) { free(lambda); return rc; }
    const double c1 = 1.0 - pow(beta1, (double)t);
    const double c2 = 1.0 - pow(beta2, (double)t);
    double sq = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : sq)
    for (int64_t j = 0; j < N; ++j) {
        double g = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            if (b[k] == 0) continue;
            g += lambda[k] * grad_at(grads[k], grad_dtype, j);
        }
        m[j] = beta1 * m[j] + (1.0 - beta1) * g;
        u[j] = beta2 * u[j] + (1.0 - beta2) * g * g;
        double mhat = m[j] / c1;
        double uhat = u[j] / c2;
        p[j] = p[j] - lr * mhat / (sqrt(uhat) + eps);
        if (g_out) g_out[j] = g;
        sq += g * g;
    }
    if (sq_out) *sq_out = sq;
    free(lambda);
    return REF_OK;
}

/*
 * Mean cross-entropy gradient of a bias-free linear-softmax classifier on one
 * worker's mini-batch (the model the weighting is checked on):
 *     Z = X W            X: [n, D] row-major, W: [D, C] row-major
 *     P = softmax over each row of Z (row maximum subtracted first)
 *     G = X^T (P - Y) / n,   Y one-hot of the labels y[i] in [0, C)
 *     loss = -(1/n) sum_i log P[i, y_i]
 * Called on a worker's rows it is that worker's mean gradient; called on the
 * concatenation of all workers' rows (n = sum b) it is the full-batch gradient
 * the weighted aggregate of Eq. 2-3 must reproduce.
 */
int ref_worker_grad(const float* X, const int32_t* y, const float* W,
                    int32_t n, int32_t D, int32_t C, double* G, double* loss) {
    if (!X || !y || !W || !G || n < 1 || D < 1 || C < 1) return REF_ERR_ARG;
    for (int32_t i = 0; i < n; ++i)
        if (y[i] < 0 || y[i] >= C) return REF_ERR_ARG;
    double* E = (double*)malloc(sizeof(double) * (size_t)n * (size_t)C);
    if (!E) return REF_ERR_ARG;
    double total = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        double* z = E + (size_t)i * C;
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int32_t d = 0; d < D; ++d)
                s += (double)X[(size_t)i * D + d] * (double)W[(size_t)d * C + c];
            z[c] = s;
        }
        double zmax = z[0];
        for (int32_t c = 1; c < C; ++c) if (z[c] > zmax) zmax = z[c];
        double den = 0.0;
        for (int32_t c = 0; c < C; ++c) den += exp(z[c] - zmax);
        total += -((z[y[i]] - zmax) - log(den));
        for (int32_t c = 0; c < C; ++c) z[c] = exp(z[c] - zmax) / den;
        z[y[i]] -= 1.0;                      /* P - Y */
    }
#pragma omp parallel for schedule(static)
    for (int32_t d = 0; d < D; ++d) {
        for (int32_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int32_t i = 0; i < n; ++i)
                s += (double)X[(size_t)i * D + d] * E[(size_t)i * C + c];
            G[(size_t)d * C + c] = s / (double)n;
        }
    }
    if (loss) *loss = total / (double)n;
    free(E);
    return REF_OK;
}

/*
 * Integer apportionment used by the controller and the static policy: real
 * targets q_k (sum S) -> integers in [lo_k, hi_k] that sum to S exactly.
 * Start from floor(q_k) clamped into the bounds; while units are missing give
 * one to the worker below its upper bound with the largest q_k - f_k; while
 * there are too many take one from the worker above its lower bound with the
 * largest f_k - q_k; ties go to the lowest index.  (The paper never says how
 * real batch sizes become integers; this is the largest-remainder rule.)
 */
static int apportion(const double* q, int32_t K, int64_t S, const int32_t* lo,
                     const int32_t* hi, int32_t* out) {
    int64_t sum_lo = 0, sum_hi = 0;
    for (int32_t k = 0; k < K; ++k) {
        int64_t l = lo ? lo[k] : 1, h = hi ? hi[k] : S;
        if (l < 0 || h < l) return REF_ERR_ARG;
        sum_lo += l;
        sum_hi += h;
    }
    if (sum_lo > S || sum_hi < S) return REF_ERR_INFEASIBLE;
    int64_t* f = (int64_t*)malloc(sizeof(int64_t) * (size_t)K);
    if (!f) return REF_ERR_ARG;
    int64_t total = 0;
    for (int32_t k = 0; k < K; ++k) {
        int64_t l = lo ? lo[k] : 1, h = hi ? hi[k] : S;
        double fl = floor(q[k]);
        int64_t x = (fl > (double)S) ? S : (fl < 0.0 ? 0 : (int64_t)fl);
        if (x < l) x = l;
        if (x > h) x = h;
        f[k] = x;
        total += x;
    }
    while (total < S) {
        int32_t best = -1;
        double best_gap = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            int64_t h = hi ? hi[k] : S;
            if (f[k] >= h) continue;
            double gap = q[k] - (double)f[k];
            if (best < 0 || gap > best_gap) { best = k; best_gap = gap; }
        }
        f[best] += 1;
        total += 1;
    }
    while (total > S) {
        int32_t best = -1;
        double best_gap = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            int64_t l = lo ? lo[k] : 1;
            if (f[k] <= l) continue;
            double gap = (double)f[k] - q[k];
            if (best < 0 || gap > best_gap) { best = k; best_gap = gap; }
        }
        f[best] -= 1;
        total -= 1;
    }
    for (int32_t k = 0; k < K; ++k) out[k] = (int32_t)f[k];
    free(f);
    return REF_OK;
}

/*
 * Real-valued controller target (before integers), exposed for the pins.
 * Section 3.3 with the sensor written through throughput, t_k = b_k / X_k:
 *     tbar   = (1/K) sum_k t_k
 *     tau_k  = t_k - tbar                       (the error)
 *     Db_k   = -X_k * tau_k                     (Eq. 4)
 *     bt_k   = b_k + kp * Db_k                  (Eq. 5; the paper has kp = 1)
 *     q_k    = bt_k * S / sum_i bt_i,  S = sum_i b_i
 * Eq. 4-5 alone do not keep the global batch S constant; the paper states
 * that invariant for variable batching (Section 3.2), so the targets are
 * rescaled to sum to S.
 */
int ref_controller_targets(const int32_t* b, const double* X, int32_t K,
                           double kp, double* q) {
    if (!b || !X || !q || K < 1) return REF_ERR_ARG;
    if (!(kp > 0.0) || !(kp <= 1.0)) return REF_ERR_ARG;
    int64_t S = 0;
    for (int32_t k = 0; k < K; ++k) {
        if (b[k] < 0) return REF_ERR_ARG;
        if (!(X[k] > 0.0) || !isfinite(X[k])) return REF_ERR_ARG;
        S += b[k];
    }
    if (S <= 0) return REF_ERR_ARG;
    double tsum = 0.0;
    for (int32_t k = 0; k < K; ++k) tsum += (double)b[k] / X[k];
    double tbar = tsum / (double)K;
    double btsum = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        double t = (double)b[k] / X[k];
        double delta = -X[k] * (t - tbar);
        q[k] = (double)b[k] + kp * delta;
        btsum += q[k];
    }
    for (int32_t k = 0; k < K; ++k) q[k] = q[k] * (double)S / btsum;
    return REF_OK;
}

/* One controller step: targets above, then the bounded integer apportionment
 * (bounds: Section 3.3.1, "Batch size bounds"; NULL means [1, S]). */
int ref_controller_step(int32_t* b, const double* X, int32_t K, double kp,
                        const int32_t* b_min, const int32_t* b_max) {
    if (!b || !X || K < 1) return REF_ERR_ARG;
    double* q = (double*)malloc(sizeof(double) * (size_t)K);
    int32_t* nb = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    if (!q || !nb) { free(q); free(nb); return REF_ERR_ARG; }
    int rc = ref_controller_targets(b, X, K, kp, q);
    if (rc == REF_OK) {
        int64_t S = 0;
        for (int32_t k = 0; k < K; ++k) S += b[k];
        rc = apportion(q, K, S, b_min, b_max, nb);
    }
    if (rc == REF_OK) memcpy(b, nb, sizeof(int32_t) * (size_t)K);
    free(q);
    free(nb);
    return rc;
}

/*
 * Static open-loop allocation (Section 3.2): b_k proportional to X_k with the
 * global batch K*b0 preserved.  The printed b0*X_k/sum X sums to b0, not to
 * the K*b0 the next sentence requires; the factor K is restored here.
 */
int ref_static_allocate(const double* X, int32_t K, int32_t b0,
                        const int32_t* b_min, const int32_t* b_max,
                        int32_t* b) {
    if (!X || !b || K < 1 || b0 < 1) return REF_ERR_ARG;
    double xsum = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        if (!(X[k] > 0.0) || !isfinite(X[k])) return REF_ERR_ARG;
        xsum += X[k];
    }
    int64_t S = (int64_t)K * b0;
    double* q = (double*)malloc(sizeof(double) * (size_t)K);
    if (!q) return REF_ERR_ARG;
    for (int32_t k = 0; k < K; ++k) q[k] = (double)S * X[k] / xsum;
    int rc = apportion(q, K, S, b_min, b_max, b);
    free(q);
    return rc;
}

/*
 * Stabilised controller (Section 3.3.1, the four-step listing), one
 * observation of per-worker iteration times t_k:
 *   1. mu_k = EWMA of t_k over the iterations since the last readjustment
 *      (first sample after a readjustment initialises it; alpha is the
 *      weight of the new sample -- the paper gives no value);
 *   2. Eq. 4-5 with mu_k in place of t_k (X_k = b_k / mu_k), gain kp,
 *      rescaled to the global batch, made integer within the bounds;
 *   3. bounds b_min <= b <= b_max (inside the apportionment).  With
 *      `adaptive` set, the upper bound also learns ("Batch size bounds"): if
 *      a worker's smoothed throughput is lower than it was at the previous
 *      readjustment although its batch was raised then (from b0 to b), its
 *      upper bound becomes b0.  Should the learnt bounds no longer admit the
 *      global batch, the user's bounds alone are used for this step;
 *   4. dead-band: readjust every worker only if max_k |b'_k - b_k| / b_k
 *      exceeds dmin (the paper uses 0.05), else keep all batch sizes.
 * State: ewma[K], n_since (samples since the last readjustment, 0 = none),
 * and for the adaptive bound prev_b[K], prev_X[K] (batch and throughput at
 * the previous readjustment; prev_X = 0 means none yet) and learnt_max[K]
 * (0 = nothing learnt).  *changed is set to 1 when the batch sizes moved.
 */
int ref_controller_observe(int32_t* b, const double* t, int32_t K, double kp,
                           double alpha, double dmin, const int32_t* b_min,
                           const int32_t* b_max, double* ewma,
                           int32_t* n_since, int32_t* changed,
                           int32_t adaptive, int32_t* prev_b, double* prev_X,
                           int32_t* learnt_max) {
    if (!b || !t || !ewma || !n_since || !changed || K < 1) return REF_ERR_ARG;
    if (adaptive && (!prev_b || !prev_X || !learnt_max)) return REF_ERR_ARG;
    if (!(alpha > 0.0) || !(alpha <= 1.0) || !(dmin >= 0.0)) return REF_ERR_ARG;
    for (int32_t k = 0; k < K; ++k)
        if (!(t[k] > 0.0) || !isfinite(t[k]) || b[k] < 1) return REF_ERR_ARG;
    for (int32_t k = 0; k < K; ++k)
        ewma[k] = (*n_since == 0) ? t[k] : alpha * t[k] + (1.0 - alpha) * ewma[k];
    *n_since += 1;
    double* X = (double*)malloc(sizeof(double) * (size_t)K);
    int32_t* nb = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    int32_t* hi = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    if (!X || !nb || !hi) { free(X); free(nb); free(hi); return REF_ERR_ARG; }
    int64_t S = 0;
    for (int32_t k = 0; k < K; ++k) { X[k] = (double)b[k] / ewma[k]; nb[k] = b[k]; S += b[k]; }
    int use_learnt = 0;
    if (adaptive) {
        for (int32_t k = 0; k < K; ++k) {
            if (prev_X[k] > 0.0 && b[k] > prev_b[k] && X[k] < prev_X[k]) {
                if (learnt_max[k] == 0 || prev_b[k] < learnt_max[k]) learnt_max[k] = prev_b[k];
            }
        }
        for (int32_t k = 0; k < K; ++k) {
            int64_t h = b_max ? b_max[k] : S;
            if (learnt_max[k] > 0 && learnt_max[k] < h) { h = learnt_max[k]; use_learnt = 1; }
            hi[k] = (int32_t)h;
        }
    }
    int rc = REF_ERR_INFEASIBLE;
    if (use_learnt) rc = ref_controller_step(nb, X, K, kp, b_min, hi);
    if (rc == REF_ERR_INFEASIBLE) {
        for (int32_t k = 0; k < K; ++k) nb[k] = b[k];
        rc = ref_controller_step(nb, X, K, kp, b_min, b_max);
    }
    *changed = 0;
    if (rc == REF_OK) {
        double worst = 0.0;
        for (int32_t k = 0; k < K; ++k) {
            double rel = fabs((double)nb[k] - (double)b[k]) / (double)b[k];
            if (rel > worst) worst = rel;
        }
        if (worst > dmin) {
            if (adaptive)
                for (int32_t k = 0; k < K; ++k) { prev_b[k] = b[k]; prev_X[k] = X[k]; }
            memcpy(b, nb, sizeof(int32_t) * (size_t)K);
            *n_since = 0;
            *changed = 1;
        }
    }
    free(X);
    free(nb);
    free(hi);
    return rc;
}

int ref_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ref_set_num_threads(int n) {
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
