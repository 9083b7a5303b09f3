/*
 * bmgd_oracle.c -- plain CPU statement of buffered mini-batch gradient descent.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct yardstick the
 * CUDA library is compared with.  It is used by the tests, by the smoke check and by
 * the benchmark's CPU-baseline leg; the product never calls it.  It shares no code,
 * header, table or helper with the CUDA sources.
 *
 * What it computes (paper, Section 2.2, Algorithm 1, inner loops over t and m):
 *
 *     for t = 1..T                       one round ("buffer epoch") over the buffer
 *       partition the buffer at random into M mini-batches
 *       for m = 1..M
 *         theta <- theta - alpha * (1/|S|) * sum_{i in S^(t,m)} grad l(X_i, Y_i; theta)   Eq. (2.1)
 *
 * with theta carried from one mini-batch, round, buffer and pass to the next.
 *
 * Per-sample gradients:
 *   least squares  (Eq. (3.1): Delta = I - alpha*Sxx, +alpha*Sxy)  (x.theta - y) x
 *   logistic       (Section 3.2.3 with b' = sigmoid)              (sigmoid(x.theta) - y) x
 *   softmax        (C-class extension; not in the paper)          outer(x, softmax(x W) - e_y)
 *
 * Readings taken where the paper is silent or at odds with itself:
 *   - no factor 2 in the gradients (Eq. (3.1) and Theorem 1's 0 < alpha < 2/lambda_1 fix it);
 *   - a ragged last mini-batch keeps its rows and is averaged by its own size;
 *   - the "random partition" of a round is a keyed bijection pi_t on [0, N0):
 *     mini-batch m is { pi_t(j) : m n <= j < min((m+1) n, N0) }.
 *
 * The bijection: round keys come from the Philox4x32-10 counter-based generator
 * (Salmon, Moraes, Dror, Shaw, SC'11), counter = (round, chain, tag, block), key = seed;
 * the keys drive an 8-round alternating Feistel network with modular addition on
 * Z_a x Z_c, a = max(32, ceil(sqrt(N0))), c = max(32, ceil(N0 / a)), so that a c >= N0 is
 * barely larger than N0; values >= N0 are walked round the cycle until they fall below N0.
 *
 * All floating point is fp64.  Stored inputs (fp64, fp32 or bf16) are widened exactly.
 * Threads (OpenMP, optional) split rows for the residuals and columns for the gradient,
 * so the result does not depend on the thread count.
 *
 * Pins (tests/test_oracle_*.py): Philox against an independent library implementation;
 * bijectivity by brute force; full-batch closed form and OLS limit; the Gram-matrix
 * recurrence Eq. (3.1)-(3.2); the stable solution below Eq. (3.3); tiny-N brute force;
 * finite differences and Newton/IRLS limits for logistic; the C = 2 softmax/logistic
 * identity; the Nesterov and Adam updates against a library optimiser fed the same gradients, and against
 * their closed forms on the first steps; the cosine rate against its printed values.  The statistical quality of the shuffle beyond the chi-square gate in the
 * tests is parity unpinned.
 */
#define _USE_MATH_DEFINES
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif
#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

enum { ORC_LINEAR = 0, ORC_LOGISTIC = 1, ORC_SOFTMAX = 2 };
enum { ORC_F64 = 0, ORC_F32 = 1, ORC_BF16 = 2 };

/* ------------------------------------------------------------------ Philox4x32-10 */

static void mulhilo32(uint32_t a, uint32_t b, uint32_t *hi, uint32_t *lo) {
    uint64_t prod = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(prod >> 32);
    *lo = (uint32_t)prod;
}

/* Ten rounds; the key is bumped by the Weyl constants between rounds. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo32(0xD2511F53u, c0, &hi0, &lo0);
        mulhilo32(0xCD9E8D57u, c2, &hi1, &lo1);
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------------------------------ shuffle */

#define ORC_SHUFFLE_TAG 0x424D4744u /* "BMGD" */
/* Narrow Feistel halves fail the chi-square gate on mini-batch co-membership, so neither
 * half of the network is ever smaller than 32 values; small buffers just walk the cycle
 * longer. */
#define ORC_MIN_HALF 32u

/* Eight Feistel round keys for (seed, chain, round). */
void orc_round_keys(uint64_t seed, uint32_t chain, uint32_t round, uint32_t keys[8]) {
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { round, chain, ORC_SHUFFLE_TAG, 0u };
    orc_philox4x32_10(ctr, key, keys);
    ctr[3] = 1u;
    orc_philox4x32_10(ctr, key, keys + 4);
}

/* The two halves of the network for a buffer of N0 rows: a = max(32, ceil(sqrt(N0))) values
 * in the high half, c = max(32, ceil(N0 / a)) in the low half.  a c >= N0, and for
 * N0 >= 1024 the excess a c - N0 is below a, i.e. a fraction of about 1/sqrt(N0). */
void orc_domain(uint32_t N0, uint32_t *a_out, uint32_t *c_out) {
    uint32_t a = (uint32_t)sqrt((double)N0);
    while ((uint64_t)a * a < N0) ++a;                       /* smallest a with a^2 >= N0 */
    while (a > 0 && (uint64_t)(a - 1) * (a - 1) >= N0) --a;
    if (a < ORC_MIN_HALF) a = ORC_MIN_HALF;
    uint32_t c = (uint32_t)(((uint64_t)N0 + a - 1) / a);
    if (c < ORC_MIN_HALF) c = ORC_MIN_HALF;
    *a_out = a;
    *c_out = c;
}

/* Round function: a keyed 32-bit hash of the other half, scaled into [0, m). */
static uint32_t feistel_g(uint32_t v, uint32_t k, uint32_t m) {
    uint32_t hi, lo;
    mulhilo32(0xD2511F53u, v + k, &hi, &lo);
    uint32_t f = hi ^ lo;
    return (uint32_t)(((uint64_t)f * (uint64_t)m) >> 32);  /* floor(f m / 2^32) */
}

/* pi(j) for j in [0, N0).  A value x of the network's domain [0, a c) is the pair
 * (L, R) = (x div c, x mod c).  Each round adds, modulo the size of one half, a function of
 * the other half: invertible, so the eight rounds are a bijection of [0, a c), and walking
 * the cycle until the value is below N0 makes it a bijection of [0, N0). */
uint32_t orc_perm_index(uint32_t j, uint32_t N0, const uint32_t keys[8]) {
    uint32_t a, c;
    orc_domain(N0, &a, &c);
    uint32_t x = j;
    do {
        uint32_t L = x / c;
        uint32_t R = x % c;
        for (int r = 0; r < 8; ++r) {
            if ((r & 1) == 0) L = (L + feistel_g(R, keys[r], a)) % a;
            else              R = (R + feistel_g(L, keys[r], c)) % c;
        }
        x = L * c + R;
    } while (x >= N0);
    return x;
}

/* The whole permutation of one round, out[j] = pi(j). */
void orc_perm(uint64_t seed, uint32_t chain, uint32_t round, uint32_t N0, uint32_t *out) {
    uint32_t keys[8];
    orc_round_keys(seed, chain, round, keys);
    for (uint32_t j = 0; j < N0; ++j) out[j] = orc_perm_index(j, N0, keys);
}

/* ------------------------------------------------------------------ stored values -> double */

static double bf16_to_double(uint16_t h) {
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static double load_x(const void *X, int xtype, int64_t idx) {
    switch (xtype) {
        case ORC_F64: return ((const double *)X)[idx];
        case ORC_F32: return (double)((const float *)X)[idx];
        default:      return bf16_to_double(((const uint16_t *)X)[idx]);
    }
}

static double sigmoid(double u) {
    if (u >= 0.0) return 1.0 / (1.0 + exp(-u));
    double e = exp(u);
    return e / (1.0 + e);
}

/* ------------------------------------------------------------------ the computation step */

/*
 * T rounds of shuffled mini-batch gradient descent over one buffer (Algorithm 1, inner loops).
 *
 *   loss       ORC_LINEAR / ORC_LOGISTIC / ORC_SOFTMAX
 *   X, xtype   buffer rows, row-major [N0][p], stored as xtype
 *   y, ytype   responses [N0]: floating (ytype = ORC_F64/ORC_F32) for linear and logistic,
 *              int32 class labels for softmax (ytype ignored)
 *   theta      [p] (or [p][C] row-major for softmax), updated in place
 *   T, n       rounds and mini-batch size; alpha the learning rate
 *   seed, chain  shuffle key; round t uses counter word t (or 0 if fixed_partition != 0)
 *   trace      if not NULL, receives theta after every step: [T*M][p*C]
 * Returns 0, or -1 on bad arguments.
 */
enum { ORC_OPT_SGD = 0, ORC_OPT_NESTEROV = 1, ORC_OPT_ADAM = 2 };
enum { ORC_LR_CONSTANT = 0, ORC_LR_COSINE = 1 };

/*
 * The update of one step, given the mini-batch's mean gradient g (Section 4.3: "the buffering idea combined
 * with" other gradient-based rules; the buffered versions differ from their baselines only in where the
 * mini-batches come from).
 *
 *   ORC_OPT_SGD       theta <- theta - lr g                                             Eq. (2.1)
 *   ORC_OPT_NESTEROV  v <- mu v - lr g;  theta <- theta + mu v - lr g                   (Nesterov's accelerated gradient in
 *                     the momentum form of Sutskever et al. 2013; mu = a; state s1 = v)
 *   ORC_OPT_ADAM      m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;  t <- t + 1;
 *                     theta <- theta - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps)   (Kingma & Ba 2014, Algorithm 1;
 *                     b1 = a, b2 = b; state s1 = m, s2 = v, *t)
 *
 * Learning rate of the j-th update of a pass of J updates (Section 4.4: alpha_{r,j} = 0.025 + 0.025 cos(j pi / TMK)
 * with initial value 0.05, j = 1..TMK in every pass r):
 *   ORC_LR_CONSTANT   lr = alpha
 *   ORC_LR_COSINE     lr = alpha (1/2 + 1/2 cos(j pi / J)),  *j_done counts the updates already taken in this pass
 */
typedef struct {
    int kind;
    double a, b, eps;
    double *s1, *s2;   /* [p*C] each, carried from call to call; may be NULL for ORC_OPT_SGD */
    int64_t *t;        /* Adam's step count, carried from call to call */
    int sched;
    int64_t period;    /* J */
    int64_t *j_done;
} orc_opt;

static void orc_apply_update(const orc_opt *o, double alpha, int q, const double *gsum, int nm, double *theta) {
    double lr = alpha;
    if (o && o->sched == ORC_LR_COSINE) {
        const int64_t j = *o->j_done + 1;
        lr = alpha * (0.5 + 0.5 * cos((double)j * M_PI / (double)o->period));
        *o->j_done = j % o->period;
    }
    const int kind = o ? o->kind : ORC_OPT_SGD;
    if (kind == ORC_OPT_SGD) {
        const double scale = lr / (double)nm;
        for (int k = 0; k < q; ++k) theta[k] -= scale * gsum[k];
    } else if (kind == ORC_OPT_NESTEROV) {
        for (int k = 0; k < q; ++k) {
            const double g = gsum[k] / (double)nm;
            o->s1[k] = o->a * o->s1[k] - lr * g;
            theta[k] += o->a * o->s1[k] - lr * g;
        }
    } else {
        *o->t += 1;
        const double c1 = 1.0 - pow(o->a, (double)*o->t), c2 = 1.0 - pow(o->b, (double)*o->t);
        for (int k = 0; k < q; ++k) {
            const double g = gsum[k] / (double)nm;
            o->s1[k] = o->a * o->s1[k] + (1.0 - o->a) * g;
            o->s2[k] = o->b * o->s2[k] + (1.0 - o->b) * g * g;
            theta[k] -= lr * (o->s1[k] / c1) / (sqrt(o->s2[k] / c2) + o->eps);
        }
    }
}

int orc_run_rounds_opt(int loss, const void *X, int xtype, const void *y, int ytype,
                       int64_t N0, int p, int C, double *theta,
                       int T, int n, double alpha, uint64_t seed, uint32_t chain,
                       int fixed_partition, double *trace, const orc_opt *opt);

int orc_run_rounds(int loss, const void *X, int xtype, const void *y, int ytype,
                   int64_t N0, int p, int C, double *theta,
                   int T, int n, double alpha, uint64_t seed, uint32_t chain,
                   int fixed_partition, double *trace) {
    return orc_run_rounds_opt(loss, X, xtype, y, ytype, N0, p, C, theta, T, n, alpha, seed, chain, fixed_partition,
                              trace, NULL);
}

/* The same with the update rule and learning-rate schedule of `opt` (NULL: Eq. (2.1) with a constant rate). */
int orc_run_rounds_opt(int loss, const void *X, int xtype, const void *y, int ytype,
                       int64_t N0, int p, int C, double *theta,
                       int T, int n, double alpha, uint64_t seed, uint32_t chain,
                       int fixed_partition, double *trace, const orc_opt *opt) {
    if (opt) {
        if (opt->kind < ORC_OPT_SGD || opt->kind > ORC_OPT_ADAM) return -1;
        if (opt->kind != ORC_OPT_SGD && !opt->s1) return -1;
        if (opt->kind == ORC_OPT_ADAM && (!opt->s2 || !opt->t)) return -1;
        if (opt->sched == ORC_LR_COSINE && (opt->period <= 0 || !opt->j_done)) return -1;
    }
    if (N0 <= 0 || N0 > 0x7FFFFFFF || p <= 0 || n <= 0 || T < 0) return -1;
    if (loss == ORC_SOFTMAX) { if (C < 2) return -1; } else C = 1;
    const int64_t M = (N0 + n - 1) / n;
    const int q = p * C;
    uint32_t *idx = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)n);
    double *res = (double *)malloc(sizeof(double) * (size_t)n * (size_t)C);
    double *g = (double *)malloc(sizeof(double) * (size_t)q);
    if (!idx || !res || !g) { free(idx); free(res); free(g); return -1; }

    int64_t step = 0;
    for (int t = 0; t < T; ++t) {
        uint32_t keys[8];
        orc_round_keys(seed, chain, fixed_partition ? 0u : (uint32_t)t, keys);
        for (int64_t m = 0; m < M; ++m) {
            const int64_t lo = m * n;
            const int64_t hi = (lo + n < N0) ? lo + n : N0;
            const int nm = (int)(hi - lo);
            for (int u = 0; u < nm; ++u) idx[u] = orc_perm_index((uint32_t)(lo + u), (uint32_t)N0, keys);

            /* residuals, one row at a time */
            #pragma omp parallel for schedule(static)
            for (int u = 0; u < nm; ++u) {
                const int64_t row = (int64_t)idx[u] * p;
                if (loss == ORC_SOFTMAX) {
                    double *z = res + (size_t)u * C;
                    for (int c = 0; c < C; ++c) z[c] = 0.0;
                    for (int j = 0; j < p; ++j) {
                        const double xj = load_x(X, xtype, row + j);
                        for (int c = 0; c < C; ++c) z[c] += xj * theta[(size_t)j * C + c];
                    }
                    double zmax = z[0];
                    for (int c = 1; c < C; ++c) if (z[c] > zmax) zmax = z[c];
                    double den = 0.0;
                    for (int c = 0; c < C; ++c) { z[c] = exp(z[c] - zmax); den += z[c]; }
                    const int label = ((const int32_t *)y)[idx[u]];
                    for (int c = 0; c < C; ++c) z[c] = z[c] / den - (c == label ? 1.0 : 0.0);
                } else {
                    double dot = 0.0;
                    for (int j = 0; j < p; ++j) dot += load_x(X, xtype, row + j) * theta[j];
                    const double yi = load_x(y, ytype, idx[u]);
                    res[u] = (loss == ORC_LOGISTIC ? sigmoid(dot) : dot) - yi;
                }
            }

            /* gradient sum, one coefficient at a time, rows in mini-batch order */
            #pragma omp parallel for schedule(static)
            for (int j = 0; j < p; ++j) {
                for (int c = 0; c < C; ++c) g[(size_t)j * C + c] = 0.0;
                for (int u = 0; u < nm; ++u) {
                    const double xj = load_x(X, xtype, (int64_t)idx[u] * p + j);
                    for (int c = 0; c < C; ++c) g[(size_t)j * C + c] += res[(size_t)u * C + c] * xj;
                }
            }

            orc_apply_update(opt, alpha, q, g, nm, theta);
            if (trace) memcpy(trace + (size_t)step * q, theta, sizeof(double) * (size_t)q);
            ++step;
        }
    }
    free(idx); free(res); free(g);
    return 0;
}

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int nthreads) {
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
}
