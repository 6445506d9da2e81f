/*
 * CPU float64 oracle for the CAME optimizer step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * optimizer computes.  Tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it; the product (the CUDA library) never does, and the two share
 * no code.
 *
 * Source of every formula: "CAME: Confidence-guided Adaptive Memory Efficient
 * Optimization", Algorithm 2 (the CAME optimizer), Algorithm 1 (Adafactor with
 * momentum), Eq. 1 (update clipping) and Eq. 2 (rank-1 non-negative
 * factorisation).  Each function below names the passage it follows and takes
 * the steps in the order the algorithm lists them.  Matrices are n x m,
 * row-major; all squares, divisions and square roots on matrices are
 * element-wise; 1_n / 1_m are all-ones vectors.
 *
 * Readings where the paper is silent (each is also a test pin or listed as
 * unpinned):
 *   - R_0 = C_0 = 0, like the listed r_0 = c_0 = m_0 = 0 (inputs of Algorithm 2).
 *   - no bias correction and no step-dependent decay: the betas are constants.
 *   - weight decay is NOT in the paper.  It is taken as decoupled decay on the
 *     previous iterate: theta_t = theta_{t-1} - eta * (m_t / sqrt(S_t) + lambda * theta_{t-1}).
 *     lambda = 0 gives Algorithm 2 exactly.  PARITY UNPINNED for lambda != 0
 *     (definition only).
 *   - vectors: the paper defines the method for matrices only.  A vector of
 *     length N takes the unfactored path: element-wise second moment v and
 *     element-wise instability S.  That is exactly what Algorithm 2 yields for
 *     an N x 1 matrix (then c = 1^T r, hence v_i = r_i, and likewise S_i = R_i),
 *     which is the pin for it.
 *
 * Pins (tests/test_oracle_pins.py): marginals of Eq. 2, exactness for rank-1
 * squared gradients, beta2 -> 0 limit, dense-EMA brute force, clip property,
 * closed-form first step, beta1 = 0 case, Algorithm 1 reduction, power-of-two
 * scale invariance, transpose and permutation equivariance, vector == N x 1.
 * Unpinned: weight decay with lambda != 0 (see above).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    double lr;            /* eta */
    double beta1, beta2, beta3;
    double eps1, eps2;
    double clip_d;        /* d */
    double weight_decay;  /* lambda, decoupled; not in the paper */
} came_oracle_hparams;

/* Optional per-call diagnostics (any pointer may be NULL). */
typedef struct {
    double sum_r;     /* 1_n^T r_t */
    double rms_u;     /* RMS(u_t) before clipping */
    double sum_R;     /* 1_n^T R_t */
} came_oracle_diag;

/* ---------------------------------------------------------------------------
 * Algorithm 2, the two factor updates (also Algorithm 1):
 *   row[i] = beta * row[i] + (1 - beta) * sum_j (X[i][j] + eps)
 *   col[j] = beta * col[j] + (1 - beta) * sum_i (X[i][j] + eps)
 * X is the matrix being factored (g^2 for r,c; the instability U for R,C).
 * The "+ eps 1_n 1_m^T" sits inside the sums, as printed.
 * ------------------------------------------------------------------------- */
void came_oracle_factor_ema(int64_t n, int64_t m, const double* X, double eps, double beta,
                            double* row, double* col)
{
    int64_t i, j;
#pragma omp parallel for private(j) schedule(static)
    for (i = 0; i < n; ++i) {
        double s = 0.0;
        for (j = 0; j < m; ++j) s += X[i * m + j] + eps;
        row[i] = beta * row[i] + (1.0 - beta) * s;
    }
    double* cs = (double*)calloc((size_t)m, sizeof(double));
    for (i = 0; i < n; ++i)
        for (j = 0; j < m; ++j) cs[j] += X[i * m + j] + eps;
    for (j = 0; j < m; ++j) col[j] = beta * col[j] + (1.0 - beta) * cs[j];
    free(cs);
}

/* ---------------------------------------------------------------------------
 * Eq. 2 / Algorithm 2 "v_t = r_t c_t / 1_n^T r_t" (and the same for S_t):
 *   out[i][j] = row[i] * col[j] / sum_i row[i]
 * Returns the normaliser 1_n^T row.
 * ------------------------------------------------------------------------- */
double came_oracle_rank1(int64_t n, int64_t m, const double* row, const double* col, double* out)
{
    int64_t i, j;
    double s = 0.0;
    for (i = 0; i < n; ++i) s += row[i];
#pragma omp parallel for private(j) schedule(static)
    for (i = 0; i < n; ++i)
        for (j = 0; j < m; ++j) out[i * m + j] = row[i] * col[j] / s;
    return s;
}

/* Eq. 1: RMS(u) = sqrt(mean of the squared components of u). */
double came_oracle_rms(int64_t count, const double* u)
{
    double s = 0.0;
    int64_t k;
    for (k = 0; k < count; ++k) s += u[k] * u[k];
    return sqrt(s / (double)count);
}

/* ---------------------------------------------------------------------------
 * One CAME step on one n x m matrix (Algorithm 2, body of the loop, in order).
 * theta, mom, r, c, R, C are updated in place.  g is read only.
 * uhat_out (n*m, may be NULL) receives the clipped update \hat u_t.
 * ------------------------------------------------------------------------- */
int came_oracle_matrix_step(int64_t n, int64_t m, double* theta, const double* g, double* mom,
                            double* r, double* c, double* R, double* C,
                            const came_oracle_hparams* hp, double* uhat_out,
                            came_oracle_diag* diag)
{
    const int64_t nm = n * m;
    int64_t k;
    double* X = (double*)malloc((size_t)nm * sizeof(double)); /* g^2, later U_t        */
    double* V = (double*)malloc((size_t)nm * sizeof(double)); /* v_t, later S_t        */
    double* u = (double*)malloc((size_t)nm * sizeof(double)); /* u_t, then \hat u_t    */
    if (!X || !V || !u) { free(X); free(V); free(u); return 1; }

    /* r_t, c_t: EMAs of the row and column sums of g_t^2 + eps1 */
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k) X[k] = g[k] * g[k];
    came_oracle_factor_ema(n, m, X, hp->eps1, hp->beta2, r, c);

    /* v_t = r_t c_t / 1_n^T r_t */
    double sum_r = came_oracle_rank1(n, m, r, c, V);

    /* u_t = g_t / sqrt(v_t) */
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k) u[k] = g[k] / sqrt(V[k]);

    /* \hat u_t = u_t / max(1, RMS(u_t) / d) */
    double rms = came_oracle_rms(nm, u);
    double denom = fmax(1.0, rms / hp->clip_d);
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k) u[k] = u[k] / denom;

    /* m_t = beta1 m_{t-1} + (1 - beta1) \hat u_t */
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k) mom[k] = hp->beta1 * mom[k] + (1.0 - hp->beta1) * u[k];

    /* U_t = (\hat u_t - m_t)^2, with the NEW m_t */
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k) { double e = u[k] - mom[k]; X[k] = e * e; }

    /* R_t, C_t: EMAs of the row and column sums of U_t + eps2 */
    came_oracle_factor_ema(n, m, X, hp->eps2, hp->beta3, R, C);

    /* S_t = R_t C_t / 1_n^T R_t */
    double sum_R = came_oracle_rank1(n, m, R, C, V);

    /* theta_t = theta_{t-1} - eta / sqrt(S_t) * m_t   (+ decoupled decay, not in the paper) */
#pragma omp parallel for schedule(static)
    for (k = 0; k < nm; ++k)
        theta[k] = theta[k] - hp->lr * (mom[k] / sqrt(V[k]) + hp->weight_decay * theta[k]);

    if (uhat_out) memcpy(uhat_out, u, (size_t)nm * sizeof(double));
    if (diag) { diag->sum_r = sum_r; diag->rms_u = rms; diag->sum_R = sum_R; }
    free(X); free(V); free(u);
    return 0;
}

/* ---------------------------------------------------------------------------
 * One CAME step on a vector of length N: the unfactored path.  v and S are
 * full-size EMAs; every line is the matrix line with the factored quantity
 * replaced by its element-wise counterpart:
 *   v_t = beta2 v + (1-beta2)(g^2 + eps1);  u = g / sqrt(v_t);  clip (Eq. 1);
 *   m_t = beta1 m + (1-beta1) \hat u;  U = (\hat u - m_t)^2;
 *   S_t = beta3 S + (1-beta3)(U + eps2);  theta -= eta (m_t / sqrt(S_t) + lambda theta).
 * no_confidence != 0 selects the alternate reading in which vectors skip the
 * confidence term (Algorithm 1's last line): theta -= eta (m_t + lambda theta);
 * S is then left untouched.
 * ------------------------------------------------------------------------- */
int came_oracle_vector_step(int64_t N, double* theta, const double* g, double* mom, double* v,
                            double* S, const came_oracle_hparams* hp, int no_confidence,
                            double* uhat_out, came_oracle_diag* diag)
{
    int64_t k;
    double* u = (double*)malloc((size_t)N * sizeof(double));
    if (!u) return 1;
    for (k = 0; k < N; ++k) v[k] = hp->beta2 * v[k] + (1.0 - hp->beta2) * (g[k] * g[k] + hp->eps1);
    for (k = 0; k < N; ++k) u[k] = g[k] / sqrt(v[k]);
    double rms = came_oracle_rms(N, u);
    double denom = fmax(1.0, rms / hp->clip_d);
    for (k = 0; k < N; ++k) u[k] = u[k] / denom;
    for (k = 0; k < N; ++k) mom[k] = hp->beta1 * mom[k] + (1.0 - hp->beta1) * u[k];
    if (no_confidence) {
        for (k = 0; k < N; ++k)
            theta[k] = theta[k] - hp->lr * (mom[k] + hp->weight_decay * theta[k]);
    } else {
        for (k = 0; k < N; ++k) {
            double e = u[k] - mom[k];
            S[k] = hp->beta3 * S[k] + (1.0 - hp->beta3) * (e * e + hp->eps2);
        }
        for (k = 0; k < N; ++k)
            theta[k] = theta[k] - hp->lr * (mom[k] / sqrt(S[k]) + hp->weight_decay * theta[k]);
    }
    if (uhat_out) memcpy(uhat_out, u, (size_t)N * sizeof(double));
    if (diag) { diag->sum_r = 0.0; diag->rms_u = rms; diag->sum_R = 0.0; }
    free(u);
    return 0;
}

/* ---------------------------------------------------------------------------
 * One step of Algorithm 1 (Adafactor with momentum) on an n x m matrix:
 * the lines of Algorithm 2 without U_t, R_t, C_t, S_t, and
 * theta_t = theta_{t-1} - eta m_t.
 * ------------------------------------------------------------------------- */
int adafactor_oracle_matrix_step(int64_t n, int64_t m, double* theta, const double* g,
                                 double* mom, double* r, double* c,
                                 const came_oracle_hparams* hp)
{
    const int64_t nm = n * m;
    int64_t k;
    double* X = (double*)malloc((size_t)nm * sizeof(double));
    double* V = (double*)malloc((size_t)nm * sizeof(double));
    double* u = (double*)malloc((size_t)nm * sizeof(double));
    if (!X || !V || !u) { free(X); free(V); free(u); return 1; }
    for (k = 0; k < nm; ++k) X[k] = g[k] * g[k];
    came_oracle_factor_ema(n, m, X, hp->eps1, hp->beta2, r, c);
    came_oracle_rank1(n, m, r, c, V);
    for (k = 0; k < nm; ++k) u[k] = g[k] / sqrt(V[k]);
    double denom = fmax(1.0, came_oracle_rms(nm, u) / hp->clip_d);
    for (k = 0; k < nm; ++k) u[k] = u[k] / denom;
    for (k = 0; k < nm; ++k) mom[k] = hp->beta1 * mom[k] + (1.0 - hp->beta1) * u[k];
    for (k = 0; k < nm; ++k)
        theta[k] = theta[k] - hp->lr * (mom[k] + hp->weight_decay * theta[k]);
    free(X); free(V); free(u);
    return 0;
}

#ifdef _OPENMP
#include <omp.h>
int came_oracle_threads(void) { return omp_get_max_threads(); }
#else
int came_oracle_threads(void) { return 1; }
#endif
