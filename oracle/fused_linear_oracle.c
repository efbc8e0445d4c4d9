/*
 * CPU oracle for the fused linear operator  Y = epilogue(act(X * W^T + b)).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * library is checked against.  It shares no code with that library and must never be
 * called from a product path.
 *
 * What it follows: the paper's fusion target is a chain of framework operators collapsed
 * into one kernel (Appendix A.1 names matmul followed by relu; Appendix B.1 names a Linear
 * layer followed by an in-register epilogue with a per-row statistic), and its correctness
 * criterion (Section 2.2, "Design of Correctness Tests") is agreement with the unfused
 * framework operators on the same inputs.  The paper prints no formula for the chain, so
 * each step below is the textbook definition of the corresponding framework operator,
 * evaluated in the order bias -> activation -> scale -> row reduction:
 *
 *   1. Z[m,n] = b[n] + sum_{k} X[m,k] * W[n,k]              (Linear; W is [N,K])
 *   2. A = act(Z)      identity | max(z,0) | 0.5 z (1+erf(z/sqrt 2))
 *                      | 0.5 z (1+tanh(sqrt(2/pi) (z + 0.044715 z^3))) | z/(1+exp(-z))
 *   3. E = scale * A
 *   4. none: Y = E;  sum: out[m] = sum_n E;  max: out[m] = max_n E;
 *      layernorm: mu = mean_n E, var = mean_n (E-mu)^2 (population variance),
 *                 Y = (E-mu)/sqrt(var+eps) * gamma[n] + beta[n]
 *      mean-gelu-residual (the chain of the Appendix B.1 case study: Linear, subtract, row
 *                 mean, GELU, residual add of the layer's input):
 *                 g[m] = gelu_erf(mean_n (E[m,n] - sub[n])),  Y[m,k] = X[m,k] + g[m]   (Y is [M,K])
 *      logsumexp: out[m] = log sum_n exp(E[m,n])   (the row statistic of a softmax; Section 4's
 *                 case study replaces block-wide reductions of exactly this max / sum pair)
 *      cross-entropy: out[m] = logsumexp_n E[m,:] - E[m, target[m]]   (Section 4: CrossEntropyLoss
 *                 per row, before the mean over rows)
 *
 * All arithmetic is IEEE double.  Inputs arrive as float (values stored as fp32 or bf16 are
 * exactly representable in float and in double).  No blocking, no reordering: k runs
 * 0..K-1, n runs 0..N-1.  Rows are independent, so `rows` may name any subset.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ACT_IDENTITY = 0, ACT_RELU = 1, ACT_GELU_ERF = 2, ACT_GELU_TANH = 3, ACT_SILU = 4 };
enum { RED_NONE = 0, RED_SUM = 1, RED_MAX = 2, RED_LAYERNORM = 3, RED_MEAN_GELU_RESIDUAL = 4,
       RED_LOGSUMEXP = 5, RED_CROSS_ENTROPY = 6 };

/* Step 2: the activation, one value at a time. */
double forge_oracle_act(int act, double z)
{
    switch (act) {
    case ACT_IDENTITY:  return z;
    case ACT_RELU:      return z > 0.0 ? z : 0.0;
    case ACT_GELU_ERF:  return 0.5 * z * (1.0 + erf(z / sqrt(2.0)));
    case ACT_GELU_TANH: return 0.5 * z * (1.0 + tanh(sqrt(2.0 / M_PI) * (z + 0.044715 * z * z * z)));
    case ACT_SILU:      return z / (1.0 + exp(-z));
    default:            return NAN;
    }
}

int forge_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * X [M,K], W [N,K], b [N] or NULL, gamma/beta [N] (layernorm only), all row-major float.
 * sub [N] (mean-gelu-residual only; NULL there means nothing is subtracted).
 * target [M] column indices (cross-entropy only).
 * rows: nrows row indices into X (NULL means rows 0..nrows-1).
 * out:  double, [nrows,N] for none/layernorm, [nrows] for sum/max/logsumexp/cross-entropy,
 *       [nrows,K] for mean-gelu-residual.
 * Returns 0, or 1 on a bad argument.
 */
int forge_oracle_fused_linear(int64_t M, int64_t N, int64_t K,
                              const float *X, const float *W, const float *b,
                              const float *gamma, const float *beta, const float *sub,
                              const int32_t *target, int act, double scale, int red, double eps,
                              const int64_t *rows, int64_t nrows, double *out)
{
    if (M <= 0 || N <= 0 || K <= 0 || nrows < 0 || !X || !W || !out) return 1;
    if (act < ACT_IDENTITY || act > ACT_SILU || red < RED_NONE || red > RED_CROSS_ENTROPY) return 1;
    if (red == RED_CROSS_ENTROPY && !target) return 1;
    if (red == RED_LAYERNORM && (!gamma || !beta)) return 1;
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t m = rows ? rows[r] : r;
        if (m < 0 || m >= M) return 1;
        if (red == RED_CROSS_ENTROPY && (target[m] < 0 || target[m] >= N)) return 1;
    }

    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nrows; ++r) {
        const int64_t m = rows ? rows[r] : r;
        double *E = (double *)malloc((size_t)N * sizeof(double));
        if (!E) {
#pragma omp atomic write
            bad = 1;
            continue;
        }

        for (int64_t n = 0; n < N; ++n) {
            double z = b ? (double)b[n] : 0.0;                       /* step 1 */
            for (int64_t k = 0; k < K; ++k)
                z += (double)X[m * K + k] * (double)W[n * K + k];
            E[n] = scale * forge_oracle_act(act, z);                 /* steps 2, 3 */
        }

        if (red == RED_NONE) {                                       /* step 4 */
            for (int64_t n = 0; n < N; ++n) out[r * N + n] = E[n];
        } else if (red == RED_SUM) {
            double s = 0.0;
            for (int64_t n = 0; n < N; ++n) s += E[n];
            out[r] = s;
        } else if (red == RED_MAX) {
            double mx = E[0];
            for (int64_t n = 1; n < N; ++n) if (E[n] > mx) mx = E[n];
            out[r] = mx;
        } else if (red == RED_LOGSUMEXP || red == RED_CROSS_ENTROPY) {
            /* log sum exp, evaluated as mx + log sum exp(E - mx) so that no term overflows */
            double mx = E[0], se = 0.0;
            for (int64_t n = 1; n < N; ++n) if (E[n] > mx) mx = E[n];
            for (int64_t n = 0; n < N; ++n) se += exp(E[n] - mx);
            out[r] = mx + log(se);
            if (red == RED_CROSS_ENTROPY) out[r] -= E[target[m]];
        } else if (red == RED_MEAN_GELU_RESIDUAL) {
            double mu = 0.0;
            for (int64_t n = 0; n < N; ++n) mu += E[n] - (sub ? (double)sub[n] : 0.0);
            mu /= (double)N;
            const double g = forge_oracle_act(ACT_GELU_ERF, mu);
            for (int64_t k = 0; k < K; ++k) out[r * K + k] = (double)X[m * K + k] + g;
        } else {
            double mu = 0.0, var = 0.0;
            for (int64_t n = 0; n < N; ++n) mu += E[n];
            mu /= (double)N;
            for (int64_t n = 0; n < N; ++n) var += (E[n] - mu) * (E[n] - mu);
            var /= (double)N;
            const double rstd = 1.0 / sqrt(var + eps);
            for (int64_t n = 0; n < N; ++n)
                out[r * N + n] = (E[n] - mu) * rstd * (double)gamma[n] + (double)beta[n];
        }
        free(E);
    }
    return bad;
}
