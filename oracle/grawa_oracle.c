/*
 * CPU ORACLE of the GRAWA / MGRAWA / LGRAWA distributed averaging update.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It is a plain, slow, float64
 * statement of what the update computes, written from the paper's equations, and
 * it shares no code with the CUDA library.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * Notation (the paper's): M workers, worker m has parameters x_m and accumulated
 * gradient G (both flat vectors of n fp32 values, read here as exact float64).
 * The flat vector is cut into K layers, layer k = [off[k], off[k+1]).
 *
 * Steps, in the paper's order:
 *   1. S[k][m]  = sum_{j in layer k} g_m[j]^2            (||G_k||_F^2 of Eq. 3 / Eq. 5)
 *   2. scores   LGRAWA  A^k_m = sqrt(S[k][m])            (Eq. 5-6)
 *               MGRAWA  A_m   = sum_k sqrt(S[k][m])      (Eq. 3: sum of per-layer Frobenius norms)
 *               GRAWA   A_m   = sqrt(sum_k S[k][m])      (Eq. 2: norm of the flattened gradient)
 *   3. weights  beta_m = (1/A_m) / sum_i (1/A_i)         (Eq. 2, Eq. 4; per layer in Eq. 7)
 *   4. centre   x_C[j] = sum_m beta_{m,k(j)} x_m[j]      (display after Eq. 2; Eq. 7 + construct)
 *   5. pull     x_m[j] <- (1-lambda) x_m[j] + lambda x_C[j], every worker, x_C from the
 *               values before the pull (the distributed update of Algorithm 1 / Algorithm 2)
 *
 * Readings where the paper is silent (both sides of the parity tests use them):
 *   - a score that is exactly 0: the limit of 1/A -> infinity.  Within one
 *     normalisation group the Z >= 1 workers with zero score share the weight
 *     equally (1/Z each), all others get 0.
 *   - a score that is not finite (NaN or +inf from NaN/Inf gradients): that worker
 *     gets weight 0 and the others are normalised among themselves; if no score of
 *     the group is finite the weights are uniform 1/M.  The flag word reports it.
 *
 * Every function here is pinned by tests/test_oracle_pins.py against closed forms,
 * hand cases, invariants and an independent numpy statement.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

enum { ORACLE_GRAWA = 0, ORACLE_MGRAWA = 1, ORACLE_LGRAWA = 2 };

/* Step 1.  S is [K][M] (row k holds the M workers' sums for layer k), index order. */
void grawa_oracle_sumsq(const float *const *grads, int M, const int64_t *off, int K, double *S)
{
    for (int k = 0; k < K; ++k)
        for (int m = 0; m < M; ++m) {
            double s = 0.0;
            for (int64_t j = off[k]; j < off[k + 1]; ++j) {
                double g = (double)grads[m][j];
                s += g * g;
            }
            S[(size_t)k * M + m] = s;
        }
}

/* Step 2.  A is [K][M] for LGRAWA, [M] for MGRAWA and GRAWA. */
void grawa_oracle_scores(const double *S, int K, int M, int variant, double *A)
{
    if (variant == ORACLE_LGRAWA) {
        for (int k = 0; k < K; ++k)
            for (int m = 0; m < M; ++m) A[(size_t)k * M + m] = sqrt(S[(size_t)k * M + m]);
    } else if (variant == ORACLE_MGRAWA) {
        for (int m = 0; m < M; ++m) {
            double a = 0.0;
            for (int k = 0; k < K; ++k) a += sqrt(S[(size_t)k * M + m]);
            A[m] = a;
        }
    } else {
        for (int m = 0; m < M; ++m) {
            double s = 0.0;
            for (int k = 0; k < K; ++k) s += S[(size_t)k * M + m];
            A[m] = sqrt(s);
        }
    }
}

/* Step 2 when the per-layer norms are given instead of gradients (the running estimates g_est of
 * the Local variants, appendix algorithm: "form x_C using the running gradient norm estimate based
 * on MGRAWA/LGRAWA policy").  N is [K][M].  LGRAWA: A^k_m = N[k][m]; MGRAWA: A_m = sum_k N[k][m]
 * (Eq. 3 with the estimate in place of ||G_k||_F); GRAWA: A_m = sqrt(sum_k N[k][m]^2). */
void grawa_oracle_scores_from_norms(const double *N, int K, int M, int variant, double *A)
{
    if (variant == ORACLE_LGRAWA) {
        for (int i = 0; i < K * M; ++i) A[i] = N[i];
    } else if (variant == ORACLE_MGRAWA) {
        for (int m = 0; m < M; ++m) {
            double a = 0.0;
            for (int k = 0; k < K; ++k) a += N[(size_t)k * M + m];
            A[m] = a;
        }
    } else {
        for (int m = 0; m < M; ++m) {
            double s = 0.0;
            for (int k = 0; k < K; ++k) s += N[(size_t)k * M + m] * N[(size_t)k * M + m];
            A[m] = sqrt(s);
        }
    }
}

/* Step 3 for one normalisation group of M scores.  Returns 1 when a non-finite
 * score was met (the fallback above was applied), else 0. */
int grawa_oracle_weights_group(const double *A, int M, double *beta)
{
    int zeros = 0, finite = 0, flagged = 0;
    for (int m = 0; m < M; ++m) {
        if (!isfinite(A[m])) flagged = 1;
        else { ++finite; if (A[m] == 0.0) ++zeros; }
    }
    if (finite == 0) {
        for (int m = 0; m < M; ++m) beta[m] = 1.0 / M;
        return flagged;
    }
    if (zeros > 0) {
        for (int m = 0; m < M; ++m) beta[m] = (isfinite(A[m]) && A[m] == 0.0) ? 1.0 / zeros : 0.0;
        return flagged;
    }
    double z = 0.0;
    for (int m = 0; m < M; ++m)
        if (isfinite(A[m])) z += 1.0 / A[m];
    for (int m = 0; m < M; ++m) beta[m] = isfinite(A[m]) ? (1.0 / A[m]) / z : 0.0;
    return flagged;
}

/* Step 3 for `groups` groups laid out [groups][M]. Returns the OR of the group flags. */
int grawa_oracle_weights(const double *A, int groups, int M, double *beta)
{
    int flagged = 0;
    for (int g = 0; g < groups; ++g)
        flagged |= grawa_oracle_weights_group(A + (size_t)g * M, M, beta + (size_t)g * M);
    return flagged;
}

/* Steps 4 and 5 on the index range [j0, j1).
 * beta: [K][M] when per_layer != 0 (layer of j found from off), else [M].
 * center_out: j1-j0 doubles (element j at center_out[j-j0]), may be NULL.
 * x_out[m]:   j1-j0 doubles each, the pulled workers, may be NULL. */
void grawa_oracle_center_pull(const float *const *x, int M, const double *beta, int per_layer,
                              const int64_t *off, int K, int64_t j0, int64_t j1, double lambda,
                              double *center_out, double *const *x_out)
{
    int k = 0;
    for (int64_t j = j0; j < j1; ++j) {
        const double *b = beta;
        if (per_layer) {
            while (k < K - 1 && j >= off[k + 1]) ++k;   /* layer that holds j (skips empty layers) */
            b = beta + (size_t)k * M;
        }
        double c = 0.0;
        for (int m = 0; m < M; ++m) c += b[m] * (double)x[m][j];
        if (center_out) center_out[j - j0] = c;
        if (x_out)
            for (int m = 0; m < M; ++m)
                x_out[m][j - j0] = (1.0 - lambda) * (double)x[m][j] + lambda * c;
    }
}

/* The whole update on the whole vector.  Outputs (any may be NULL except beta):
 * S [K][M], A and beta ([K][M] for LGRAWA else [M]), center n doubles, x_out[m] n doubles.
 * Returns the non-finite flag of step 3. */
int grawa_oracle_step(const float *const *x, const float *const *grads, int64_t n, int M,
                      const int64_t *off, int K, int variant, double lambda,
                      double *S, double *A, double *beta, double *center_out, double *const *x_out)
{
    (void)n;
    grawa_oracle_sumsq(grads, M, off, K, S);
    grawa_oracle_scores(S, K, M, variant, A);
    int groups = (variant == ORACLE_LGRAWA) ? K : 1;
    int flagged = grawa_oracle_weights(A, groups, M, beta);
    grawa_oracle_center_pull(x, M, beta, variant == ORACLE_LGRAWA, off, K, 0, off[K], lambda,
                             center_out, x_out);
    return flagged;
}

/* Proximity search step of the local phase (the "Prox." update of Algorithm 1 / 2):
 * x_m[j] <- (1 - mu/tau) x_m[j] + (mu/tau) x_C[j], with the stored centre. */
void grawa_oracle_prox(const float *const *x, int M, const float *center, int64_t n,
                       double mu_over_tau, double *const *x_out)
{
    for (int m = 0; m < M; ++m)
        for (int64_t j = 0; j < n; ++j)
            x_out[m][j] = (1.0 - mu_over_tau) * (double)x[m][j] + mu_over_tau * (double)center[j];
}

/* Running gradient-norm estimate of the "local" variants (appendix on Local GRAWA):
 * g_mvg <- gamma g_mvg + (1-gamma) g_cur ; g_est <- gamma g_mvg / (1 - gamma^t), taken literally,
 * t counted from 1.  Vectors of K entries. */
void grawa_oracle_norm_ema(double *g_mvg, const double *g_cur, int K, double gamma, int64_t t,
                           double *g_est)
{
    double corr = 1.0 - pow(gamma, (double)t);
    for (int k = 0; k < K; ++k) {
        g_mvg[k] = gamma * g_mvg[k] + (1.0 - gamma) * g_cur[k];
        g_est[k] = gamma * g_mvg[k] / corr;
    }
}
