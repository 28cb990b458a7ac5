/*
 * fp64 CPU oracle for the language-model loss head: projection onto the vocabulary followed by softmax
 * cross-entropy.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file; it shares no code, header,
 * table or constant with the CUDA sources.
 *
 * What it computes is the plain definition of the chain the paper fuses (Section 4.1, case study "Fusing a
 * Reduction into a Contraction Epilogue"; Section 6.1, "Fused Loss Head"): logits by one contraction, then a
 * row maximum and a row sum of exponentials along the vocabulary axis, then the negative log-likelihood of
 * the target.  The paper's kernel groups the maximum and the sum per N tile of the contraction and merges
 * the partial (max, sum) pairs afterwards, rescaling each sum by the exponential of the difference of the
 * maxima; that grouping reaches exactly this result and is NOT replayed here (no tiles, no partials, no
 * merge, no base 2):
 *
 *   z_in   = sum_k X[i,k] W[n,k]                         logits, i < M rows, n < N vocabulary entries
 *   m_i    = max_n z_in ;  LSE_i = m_i + ln sum_n exp(z_in - m_i)          (natural log)
 *   loss_i = LSE_i - z_{i, target_i}          for 0 <= target_i < N;  0 for any other target (ignored row)
 *
 * Everything is double precision; every sum runs in index order.  Rows are independent and are spread over
 * OpenMP threads, so results do not depend on the thread count.
 *
 * Layout: X [M, K], W [N, K] (both K fastest), targets [M] int32, logits [M, N] (may be NULL), lse [M],
 * loss [M].  All pointers are host pointers owned by the caller.  Return 0 = ok, -1 = bad argument.
 */
#include <math.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_lmhead_fwd(const double *X, const double *W, const int *targets, double *logits, double *lse,
                      double *loss, int M, int N, int K)
{
    if (!X || !W || !targets || !lse || !loss || M <= 0 || N <= 0 || K <= 0) return -1;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < M; ++i) {
        const double *x = X + (size_t)i * K;
        const int t = targets[i];
        double m = 0.0, z_t = 0.0;
        /* first pass: logits of the row, their maximum, the target's logit */
        for (int n = 0; n < N; ++n) {
            const double *w = W + (size_t)n * K;
            double z = 0.0;
            for (int k = 0; k < K; ++k) z += x[k] * w[k];
            if (logits) logits[(size_t)i * N + n] = z;
            if (n == 0 || z > m) m = z;
            if (n == t) z_t = z;
        }
        /* second pass: sum of exponentials relative to the maximum */
        double l = 0.0;
        for (int n = 0; n < N; ++n) {
            double z;
            if (logits) {
                z = logits[(size_t)i * N + n];
            } else {
                const double *w = W + (size_t)n * K;
                z = 0.0;
                for (int k = 0; k < K; ++k) z += x[k] * w[k];
            }
            l += exp(z - m);
        }
        if (!(l > 0.0)) {
#pragma omp atomic write
            bad = 1;
        }
        lse[i] = m + log(l);
        loss[i] = (t >= 0 && t < N) ? lse[i] - z_t : 0.0;
    }
    return bad ? -1 : 0;
}
