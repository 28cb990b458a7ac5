/*
 * fp64 CPU oracle for masked softmax attention and its analytic gradients.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file; it exists so that the
 * CUDA kernels can be compared with the plain mathematical definition.  It shares no code, header,
 * table or constant with the CUDA sources.
 *
 * What it computes is the definition the paper's fused kernels reformulate exactly (Section 4.2,
 * "Building the Online Softmax": scores = scale * Q K^T, causal mask keeps keys j <= i, softmax over
 * the kept keys, output = P V, log-sum-exp saved per row; "The Backward Pass": dQ reduces over keys,
 * dK and dV reduce over queries, P recomputed rather than stored).  The online/base-2/tile-clamped
 * form of the listing in Section 4.2 is *not* replayed here: the paper states those rewrites are
 * bit-identical reformulations, so the oracle is the textbook definition written out:
 *
 *   s_ij  = scale * sum_d Q[i,d] K[j,d]                       j in A_i  (A_i = {0..i} causal, else all)
 *   m_i   = max_j s_ij ;  l_i = sum_j exp(s_ij - m_i) ;  LSE_i = m_i + ln l_i      (natural log)
 *   P_ij  = exp(s_ij - LSE_i) ;  O_i = sum_j P_ij V_j
 *   dP_ij = sum_d dO[i,d] V[j,d] ;  Delta_i = sum_j P_ij dP_ij   (softmax Jacobian row term)
 *   dS_ij = P_ij (dP_ij - Delta_i)
 *   dV_j  = sum_i P_ij dO_i ;  dQ_i = scale sum_j dS_ij K_j ;  dK_j = scale sum_i dS_ij Q_i
 *
 * i.e. the gradient of L = sum(O * dO) with dO held constant.  Everything is double precision, no
 * tiling, no running rescale, no sentinel mask values (masked keys are simply not in the index set).
 * One row of scores is held at a time, never a T x T matrix.  Heads are independent and are spread
 * over OpenMP threads; within a head every sum runs in a fixed serial order, so results do not depend
 * on the thread count.
 *
 * Layout of every tensor: [B, H, T, D] contiguous (D fastest); row vectors [B, H, T].
 * All pointers are host pointers owned by the caller.  Return value 0 = ok, -1 = bad argument,
 * -2 = out of memory.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int n_keys_of_row(int i, int T, int causal) { return causal ? i + 1 : T; }

/* s[j] = scale * <q_i, K_j> for j < n */
static void score_row(const double *q_i, const double *K, int n, int D, double scale, double *s)
{
    for (int j = 0; j < n; ++j) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += q_i[d] * K[(size_t)j * D + d];
        s[j] = scale * acc;
    }
}

/* In place: s[j] -> P[j] = exp(s[j] - LSE); returns LSE = m + ln(sum exp(s - m)). */
static double softmax_row(double *s, int n)
{
    double m = s[0];
    for (int j = 1; j < n; ++j) if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int j = 0; j < n; ++j) l += exp(s[j] - m);
    double lse = m + log(l);
    for (int j = 0; j < n; ++j) s[j] = exp(s[j] - lse);
    return lse;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Forward: O [B,H,T,D], LSE [B,H,T]. */
int oracle_attn_fwd(const double *Q, const double *K, const double *V, double *O, double *LSE,
                    int B, int H, int T, int D, double scale, int causal)
{
    if (!Q || !K || !V || !O || !LSE || B <= 0 || H <= 0 || T <= 0 || D <= 0) return -1;
    int status = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        const double *q = Q + (size_t)bh * T * D, *k = K + (size_t)bh * T * D, *v = V + (size_t)bh * T * D;
        double *o = O + (size_t)bh * T * D, *lse = LSE + (size_t)bh * T;
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        if (!p) { status = -2; continue; }
        for (int i = 0; i < T; ++i) {
            int n = n_keys_of_row(i, T, causal);
            score_row(q + (size_t)i * D, k, n, D, scale, p);
            lse[i] = softmax_row(p, n);
            for (int d = 0; d < D; ++d) o[(size_t)i * D + d] = 0.0;
            for (int j = 0; j < n; ++j)
                for (int d = 0; d < D; ++d) o[(size_t)i * D + d] += p[j] * v[(size_t)j * D + d];
        }
        free(p);
    }
    return status;
}

/* Probabilities of ONE head, dense [T,T] (zeros outside A_i).  For invariants on small T. */
int oracle_attn_probs(const double *Q, const double *K, double *P, int T, int D, double scale, int causal)
{
    if (!Q || !K || !P || T <= 0 || D <= 0) return -1;
    for (int i = 0; i < T; ++i) {
        int n = n_keys_of_row(i, T, causal);
        double *row = P + (size_t)i * T;
        score_row(Q + (size_t)i * D, K, n, D, scale, row);
        (void)softmax_row(row, n);
        for (int j = n; j < T; ++j) row[j] = 0.0;
    }
    return 0;
}

/* Backward: dQ, dK, dV [B,H,T,D] and Delta [B,H,T] from Q, K, V, dO alone (P is recomputed from
 * the definition, not from a stored LSE). */
int oracle_attn_bwd(const double *Q, const double *K, const double *V, const double *dO,
                    double *dQ, double *dK, double *dV, double *Delta,
                    int B, int H, int T, int D, double scale, int causal)
{
    if (!Q || !K || !V || !dO || !dQ || !dK || !dV || !Delta || B <= 0 || H <= 0 || T <= 0 || D <= 0)
        return -1;
    int status = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        size_t off = (size_t)bh * T * D;
        const double *q = Q + off, *k = K + off, *v = V + off, *go = dO + off;
        double *gq = dQ + off, *gk = dK + off, *gv = dV + off, *delta = Delta + (size_t)bh * T;
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        double *dp = (double *)malloc(sizeof(double) * (size_t)T);
        if (!p || !dp) { free(p); free(dp); status = -2; continue; }
        memset(gq, 0, sizeof(double) * (size_t)T * D);
        memset(gk, 0, sizeof(double) * (size_t)T * D);
        memset(gv, 0, sizeof(double) * (size_t)T * D);
        for (int i = 0; i < T; ++i) {
            int n = n_keys_of_row(i, T, causal);
            const double *q_i = q + (size_t)i * D, *go_i = go + (size_t)i * D;
            score_row(q_i, k, n, D, scale, p);
            (void)softmax_row(p, n);
            /* dP_ij = <dO_i, V_j> (no scale: O = P V) */
            score_row(go_i, v, n, D, 1.0, dp);
            double dl = 0.0;
            for (int j = 0; j < n; ++j) dl += p[j] * dp[j];
            delta[i] = dl;
            for (int j = 0; j < n; ++j) {
                double ds = p[j] * (dp[j] - dl);
                for (int d = 0; d < D; ++d) {
                    gv[(size_t)j * D + d] += p[j] * go_i[d];
                    gq[(size_t)i * D + d] += scale * ds * k[(size_t)j * D + d];
                    gk[(size_t)j * D + d] += scale * ds * q_i[d];
                }
            }
        }
        free(p);
        free(dp);
    }
    return status;
}
