/*
 * VeLoRA fp64 CPU oracle  --  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, double-precision restatement of the rank-1 sub-token
 * projection of a linear layer's input (arxiv 2405.17991, Section 3.1),
 * written from the paper's definitions.  It shares no source, header,
 * table or helper with the CUDA library and is only ever called from the
 * tests, from the smoke check and from the benchmark's CPU-baseline leg.
 *
 * Symbols (the paper's "M" is a LENGTH; here, to avoid the clash):
 *   N     tokens (batch and sequence flattened)
 *   D     feature width of the linear's input
 *   Dsub  sub-token length              (the paper's M, Section 3.1)
 *   M     sub-tokens per token = ceil(D / Dsub)   (the paper's D/M)
 *   O     output width of the linear
 *
 * Reading taken where the paper is silent: when Dsub does not divide D the
 * last sub-token of a token is the remaining D - (M-1)*Dsub entries followed
 * by zeros (the paper's group() is a reshape and assumes divisibility).
 *
 * Every array is row-major with an explicit leading dimension, all double.
 * Loops follow the definitions one to one: no blocking, no fusion.  The
 * only concession to run time is an OpenMP "parallel for" over an outer
 * index whose iterations are independent (never over a summation index),
 * so results do not depend on the thread count.
 *
 * Pins (tests/test_oracle_pins.py): unit norm, orthogonal residual,
 * Pythagoras, exact cases (multiples of v, Dsub = 1, constant input),
 * idempotence, linearity, sign flip, sum(Z) = ||s||, brute force vs factored
 * weight gradient, the closed form dW = (dY^T X)(I (x) v v^T) against
 * numpy's matmul, and textbook GEMMs against numpy's matmul; the running
 * average against init_v (rho = 1; rho = 1/t over equal batches) and its
 * fixed points.  No function here is "parity unpinned"; what the running
 * average's formula should be is a reading of the paper, stated above it.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_DEGENERATE_V 5

int velora_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int64_t count_subtokens(int64_t D, int64_t Dsub)
{
    return (D + Dsub - 1) / Dsub;
}

/*
 * Initialisation of v: "the average of sub-tokens from the first batch"
 * (Section 3.2, "Cheap initialisation strategies"), made "a fixed vector of
 * unit length" (Section 3.1, definition of proj_v).
 *   s[j] = sum_n sum_m Xp[n, m*Dsub + j],   v = s / ||s||_2
 * Xp is X zero-extended to width M*Dsub.  Dividing s by the sub-token count
 * first would cancel in the normalisation, so it is not done.
 * s_out (may be NULL) receives the un-normalised sum, norm_out its length.
 * Returns ORACLE_DEGENERATE_V (v untouched) if ||s|| is zero or not finite.
 */
int velora_oracle_init_v(const double *X, int64_t N, int64_t D, int64_t ldx, int64_t Dsub,
                         double *v, double *s_out, double *norm_out)
{
    if (!X || !v || N < 0 || D < 1 || Dsub < 1 || Dsub > D || ldx < D) return ORACLE_BAD_ARG;
    if (Dsub > 4096) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    double s[4096];
    for (int64_t j = 0; j < Dsub; ++j) s[j] = 0.0;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t m = 0; m < M; ++m)
            for (int64_t j = 0; j < Dsub; ++j) {
                const int64_t d = m * Dsub + j;
                if (d < D) s[j] += X[n * ldx + d];
            }
    double sq = 0.0;
    for (int64_t j = 0; j < Dsub; ++j) sq += s[j] * s[j];
    const double norm = sqrt(sq);
    if (s_out) for (int64_t j = 0; j < Dsub; ++j) s_out[j] = s[j];
    if (norm_out) *norm_out = norm;
    if (!(norm > 0.0) || !isfinite(norm)) return ORACLE_DEGENERATE_V;
    for (int64_t j = 0; j < Dsub; ++j) v[j] = s[j] / norm;
    return ORACLE_OK;
}

/*
 * Running-average variant of the initialisation (Section 5, "Initialisation
 * strategy": the "Running average" row of the ablation table).  The paper
 * names the variant and gives no formula; the reading taken here is an
 * exponential average of the per-batch sub-token means, re-normalised:
 *   mean[j] = (1 / (N*M)) * sum_n sum_m Xp[n, m*Dsub + j]
 *   a'[j]   = (1 - rho) * a[j] + rho * mean[j]          (rho == 1: a' = mean, a is not read)
 *   v       = a' / ||a'||_2
 * rho = 1 follows every incoming batch; rho = 1/t at the t-th batch makes a'
 * the mean of everything seen so far (equal-size batches), whose direction is
 * the fixed-average v of velora_oracle_init_v on the concatenated batches.
 * Returns ORACLE_DEGENERATE_V (a_out, v untouched) if ||a'|| is zero or not finite.
 */
int velora_oracle_update_v(const double *X, int64_t N, int64_t D, int64_t ldx, int64_t Dsub,
                           double rho, const double *a, double *a_out, double *v)
{
    if (!X || !v || !a_out || N < 1 || D < 1 || Dsub < 1 || Dsub > D || ldx < D) return ORACLE_BAD_ARG;
    if (Dsub > 4096 || (rho != 1.0 && !a)) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    double an[4096];
    for (int64_t j = 0; j < Dsub; ++j) {
        double sum = 0.0;
        for (int64_t n = 0; n < N; ++n)
            for (int64_t m = 0; m < M; ++m) {
                const int64_t d = m * Dsub + j;
                if (d < D) sum += X[n * ldx + d];
            }
        const double mean = sum / ((double)N * (double)M);
        an[j] = (rho == 1.0) ? mean : (1.0 - rho) * a[j] + rho * mean;
    }
    double sq = 0.0;
    for (int64_t j = 0; j < Dsub; ++j) sq += an[j] * an[j];
    const double norm = sqrt(sq);
    if (!(norm > 0.0) || !isfinite(norm)) return ORACLE_DEGENERATE_V;
    for (int64_t j = 0; j < Dsub; ++j) {
        a_out[j] = an[j];
        v[j] = an[j] / norm;
    }
    return ORACLE_OK;
}

/*
 * compress(z; v) = z . v for every sub-token (Section 3.1, Eq. 1):
 *   Z[n, m] = sum_{j < Dsub} Xp[n, m*Dsub + j] * v[j]
 */
int velora_oracle_compress(const double *X, int64_t N, int64_t D, int64_t ldx, int64_t Dsub,
                           const double *v, double *Z, int64_t ldz)
{
    if (!X || !v || !Z || N < 0 || D < 1 || Dsub < 1 || Dsub > D || ldx < D) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    if (ldz < M) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t m = 0; m < M; ++m) {
            double dot = 0.0;
            for (int64_t j = 0; j < Dsub; ++j) {
                const int64_t d = m * Dsub + j;
                if (d < D) dot += X[n * ldx + d] * v[j];
            }
            Z[n * ldz + m] = dot;
        }
    return ORACLE_OK;
}

/*
 * reconstruct(z_p; v) = z_p . v^T followed by ungroup (Section 3.1, Eq. 2):
 *   Xhat[n, m*Dsub + j] = Z[n, m] * v[j]      for m*Dsub + j < D
 */
int velora_oracle_reconstruct(const double *Z, int64_t ldz, int64_t N, int64_t D, int64_t Dsub,
                              const double *v, double *Xhat, int64_t ldxhat)
{
    if (!Z || !v || !Xhat || N < 0 || D < 1 || Dsub < 1 || Dsub > D || ldxhat < D) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    if (ldz < M) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t m = 0; m < M; ++m)
            for (int64_t j = 0; j < Dsub; ++j) {
                const int64_t d = m * Dsub + j;
                if (d < D) Xhat[n * ldxhat + d] = Z[n * ldz + m] * v[j];
            }
    return ORACLE_OK;
}

/*
 * Weight gradient, the plain definition (Algorithm 1, backward:
 * grad_weight = grad_output^T @ input, with input = ungroup(reconstruct(z, v))):
 *   dW[o, d] = beta * dW0[o, d] + sum_n dY[n, o] * Xhat[n, d]
 * Xhat[n, d] is formed on the spot from Z and v exactly as in
 * velora_oracle_reconstruct.  This form is the authoritative one.
 */
int velora_oracle_weight_grad_bruteforce(const double *dY, int64_t N, int64_t O, int64_t lddy,
                                         const double *Z, int64_t ldz, const double *v,
                                         int64_t D, int64_t Dsub,
                                         double *dW, int64_t lddw, int beta)
{
    if (!dY || !Z || !v || !dW || N < 0 || O < 1 || D < 1 || Dsub < 1 || Dsub > D) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    if (lddy < O || ldz < M || lddw < D || (beta != 0 && beta != 1)) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < O; ++o)
        for (int64_t d = 0; d < D; ++d) {
            const int64_t m = d / Dsub;
            const int64_t j = d - m * Dsub;
            double acc = 0.0;
            for (int64_t n = 0; n < N; ++n) {
                const double xhat = Z[n * ldz + m] * v[j];
                acc += dY[n * lddy + o] * xhat;
            }
            dW[o * lddw + d] = (beta ? dW[o * lddw + d] : 0.0) + acc;
        }
    return ORACLE_OK;
}

/*
 * Weight gradient, rank-1 factored form.  Because Xhat[n, m*Dsub+j] =
 * Z[n,m] v[j], the sum over tokens factors:
 *   P[o, m] = sum_n dY[n, o] * Z[n, m],   dW[o, m*Dsub + j] = beta*dW0 + P[o, m] * v[j]
 * (the paper prints the Dsub = D case, Section 3.2 "Connection to parameter
 * efficient fine-tuning": dL/dW ~ g v v^T).  Coded separately from the brute
 * force above; the tests prove the two equal on small inputs, after which
 * this one serves where brute force is too slow.  P_out (may be NULL) gets P.
 */
int velora_oracle_weight_grad_factored(const double *dY, int64_t N, int64_t O, int64_t lddy,
                                       const double *Z, int64_t ldz, const double *v,
                                       int64_t D, int64_t Dsub,
                                       double *dW, int64_t lddw, int beta, double *P_out)
{
    if (!dY || !Z || !v || !dW || N < 0 || O < 1 || D < 1 || Dsub < 1 || Dsub > D) return ORACLE_BAD_ARG;
    const int64_t M = count_subtokens(D, Dsub);
    if (lddy < O || ldz < M || lddw < D || (beta != 0 && beta != 1)) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < O; ++o)
        for (int64_t m = 0; m < M; ++m) {
            double p = 0.0;
            for (int64_t n = 0; n < N; ++n) p += dY[n * lddy + o] * Z[n * ldz + m];
            if (P_out) P_out[o * M + m] = p;
            for (int64_t j = 0; j < Dsub; ++j) {
                const int64_t d = m * Dsub + j;
                if (d < D) dW[o * lddw + d] = (beta ? dW[o * lddw + d] : 0.0) + p * v[j];
            }
        }
    return ORACLE_OK;
}

/*
 * Forward of the linear layer, unchanged by the method (Algorithm 1, forward).
 * The listing's "input @ weight" together with its backward lines fixes the
 * weight as W[O, D] applied as X W^T:
 *   Y[n, o] = sum_d X[n, d] * W[o, d]
 */
int velora_oracle_linear_forward(const double *X, int64_t N, int64_t D, int64_t ldx,
                                 const double *W, int64_t O, int64_t ldw,
                                 double *Y, int64_t ldy)
{
    if (!X || !W || !Y || N < 0 || D < 1 || O < 1 || ldx < D || ldw < D || ldy < O) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t o = 0; o < O; ++o) {
            double acc = 0.0;
            for (int64_t d = 0; d < D; ++d) acc += X[n * ldx + d] * W[o * ldw + d];
            Y[n * ldy + o] = acc;
        }
    return ORACLE_OK;
}

/*
 * Input gradient (Algorithm 1, backward: grad_input = grad_output @ weight);
 * exact, it never sees Z or v:
 *   dX[n, d] = sum_o dY[n, o] * W[o, d]
 */
int velora_oracle_input_grad(const double *dY, int64_t N, int64_t O, int64_t lddy,
                             const double *W, int64_t D, int64_t ldw,
                             double *dX, int64_t lddx)
{
    if (!dY || !W || !dX || N < 0 || D < 1 || O < 1 || lddy < O || ldw < D || lddx < D) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int64_t o = 0; o < O; ++o) acc += dY[n * lddy + o] * W[o * ldw + d];
            dX[n * lddx + d] = acc;
        }
    return ORACLE_OK;
}
