/* CPU fp64 oracle for HilbertA masked attention.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain definition of what Algorithm 1 computes: for one query row i the
 * allowed keys are those j with  M[i,j] = global(i) or global(j) or
 * (i, j image tokens of the same slid tile)  (Sec. 3.2, Sec. 3.3, Appendix A),
 * and the output is  sum_j softmax_j(s * <q_i, k_j>) v_j  over those keys.
 * Two passes per row (logits and their maximum, then exponentials), double
 * accumulation, no blocking, no online rescaling.  Inputs are float32 arrays
 * (which hold bf16 and fp32 values exactly) widened to double element by
 * element.  Nothing here is shared with, or called by, the CUDA library.
 *
 * Layout: q, k, v are [BH, S, D] contiguous in the ORIGINAL token order;
 * out is [BH, n_rows, D] double; lse (optional, may be NULL) is [BH, n_rows]
 * with lse = max + ln(sum exp) of the scaled logits.
 * rows[n] lists the query rows wanted (all of them for a full result).
 * Returns the number of worker threads used, or -1 on allocation failure.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int allowed(const uint8_t *is_global, const int32_t *group, int i, int j) {
    if (is_global[i] || is_global[j]) return 1;
    return group[i] >= 0 && group[j] >= 0 && group[i] == group[j];
}

int hilberta_oracle_attention_rows(const float *q, const float *k, const float *v,
                                   double *out, double *lse,
                                   int BH, int S, int D,
                                   const uint8_t *is_global, const int32_t *group,
                                   const int32_t *rows, int n_rows, double scale) {
    int threads = 1;
    int failed = 0;
    long total = (long)BH * n_rows;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
#pragma omp parallel
    {
        double *logit = (double *)malloc(sizeof(double) * (size_t)S);
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
        if (!logit || !acc) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (long w = 0; w < total; ++w) {
                int bh = (int)(w / n_rows);
                int n = (int)(w % n_rows);
                int i = rows[n];
                const float *qi = q + ((size_t)bh * S + i) * D;
                const float *kb = k + (size_t)bh * S * D;
                const float *vb = v + (size_t)bh * S * D;
                double m = -INFINITY;
                for (int j = 0; j < S; ++j) {
                    if (!allowed(is_global, group, i, j)) continue;
                    const float *kj = kb + (size_t)j * D;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += (double)qi[d] * (double)kj[d];
                    logit[j] = scale * dot;
                    if (logit[j] > m) m = logit[j];
                }
                double l = 0.0;
                for (int d = 0; d < D; ++d) acc[d] = 0.0;
                for (int j = 0; j < S; ++j) {
                    if (!allowed(is_global, group, i, j)) continue;
                    double p = exp(logit[j] - m);
                    const float *vj = vb + (size_t)j * D;
                    l += p;
                    for (int d = 0; d < D; ++d) acc[d] += p * (double)vj[d];
                }
                double *o = out + ((size_t)bh * n_rows + n) * D;
                for (int d = 0; d < D; ++d) o[d] = acc[d] / l;
                if (lse) lse[(size_t)bh * n_rows + n] = m + log(l);
            }
        }
        free(logit);
        free(acc);
    }
    return failed ? -1 : threads;
}

/* Backward of the same definition (the paper fine-tunes through its kernel,
 * Sec. 4.1, and prints no backward formulas; this is the plain derivative).
 * With P_ij the softmax weights of row i over its allowed keys and
 * dP_ij = <dO_i, v_j>:
 *     delta_i = sum_j P_ij dP_ij,   dS_ij = P_ij (dP_ij - delta_i),
 *     dQ_i = s sum_j dS_ij k_j,   dK_j = s sum_i dS_ij q_i,   dV_j = sum_i P_ij dO_i.
 * Pass 1 walks every query row (its log-sum-exp and delta are needed by every
 * key column it touches) and writes dQ for the rows listed in `rows`;
 * pass 2 walks the key columns listed in `cols` and, for each, every query row
 * allowed to see it.  dq is [BH, n_rows, D], dk and dv are [BH, n_cols, D],
 * all double; any of the three may be NULL.  Returns the thread count or -1.
 */
int hilberta_oracle_attention_backward(const float *q, const float *k, const float *v, const float *dout,
                                       double *dq, double *dk, double *dv,
                                       int BH, int S, int D,
                                       const uint8_t *is_global, const int32_t *group,
                                       const int32_t *rows, int n_rows,
                                       const int32_t *cols, int n_cols, double scale) {
    int threads = 1;
    int failed = 0;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
    double *lse = (double *)malloc(sizeof(double) * (size_t)BH * S);
    double *delta = (double *)malloc(sizeof(double) * (size_t)BH * S);
    int32_t *row_slot = (int32_t *)malloc(sizeof(int32_t) * (size_t)S);
    if (!lse || !delta || !row_slot) {
        free(lse); free(delta); free(row_slot);
        return -1;
    }
    for (int i = 0; i < S; ++i) row_slot[i] = -1;
    for (int n = 0; n < n_rows; ++n) row_slot[rows[n]] = n;
    long total = (long)BH * S;
#pragma omp parallel
    {
        double *logit = (double *)malloc(sizeof(double) * (size_t)S);
        double *dp = (double *)malloc(sizeof(double) * (size_t)S);
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
        if (!logit || !dp || !acc) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (long w = 0; w < total; ++w) {
                int bh = (int)(w / S);
                int i = (int)(w % S);
                const float *qi = q + ((size_t)bh * S + i) * D;
                const float *doi = dout + ((size_t)bh * S + i) * D;
                const float *kb = k + (size_t)bh * S * D;
                const float *vb = v + (size_t)bh * S * D;
                double m = -INFINITY;
                for (int j = 0; j < S; ++j) {
                    if (!allowed(is_global, group, i, j)) continue;
                    const float *kj = kb + (size_t)j * D;
                    const float *vj = vb + (size_t)j * D;
                    double dot = 0.0, dpv = 0.0;
                    for (int d = 0; d < D; ++d) {
                        dot += (double)qi[d] * (double)kj[d];
                        dpv += (double)doi[d] * (double)vj[d];
                    }
                    logit[j] = scale * dot;
                    dp[j] = dpv;
                    if (logit[j] > m) m = logit[j];
                }
                double l = 0.0;
                for (int j = 0; j < S; ++j)
                    if (allowed(is_global, group, i, j)) l += exp(logit[j] - m);
                double L = m + log(l);
                double dl = 0.0;
                for (int j = 0; j < S; ++j)
                    if (allowed(is_global, group, i, j)) dl += exp(logit[j] - L) * dp[j];
                lse[(size_t)bh * S + i] = L;
                delta[(size_t)bh * S + i] = dl;
                if (dq && row_slot[i] >= 0) {
                    for (int d = 0; d < D; ++d) acc[d] = 0.0;
                    for (int j = 0; j < S; ++j) {
                        if (!allowed(is_global, group, i, j)) continue;
                        double ds = exp(logit[j] - L) * (dp[j] - dl);
                        const float *kj = kb + (size_t)j * D;
                        for (int d = 0; d < D; ++d) acc[d] += ds * (double)kj[d];
                    }
                    double *o = dq + ((size_t)bh * n_rows + row_slot[i]) * D;
                    for (int d = 0; d < D; ++d) o[d] = scale * acc[d];
                }
            }
        }
        free(logit); free(dp); free(acc);
    }
    if (!failed && (dk || dv)) {
        long total2 = (long)BH * n_cols;
#pragma omp parallel
        {
            double *ak = (double *)malloc(sizeof(double) * (size_t)D);
            double *av = (double *)malloc(sizeof(double) * (size_t)D);
            if (!ak || !av) {
#pragma omp atomic write
                failed = 1;
            } else {
#pragma omp for schedule(dynamic, 4)
                for (long w = 0; w < total2; ++w) {
                    int bh = (int)(w / n_cols);
                    int n = (int)(w % n_cols);
                    int j = cols[n];
                    const float *kj = k + ((size_t)bh * S + j) * D;
                    const float *vj = v + ((size_t)bh * S + j) * D;
                    for (int d = 0; d < D; ++d) ak[d] = av[d] = 0.0;
                    for (int i = 0; i < S; ++i) {
                        if (!allowed(is_global, group, i, j)) continue;
                        const float *qi = q + ((size_t)bh * S + i) * D;
                        const float *doi = dout + ((size_t)bh * S + i) * D;
                        double dot = 0.0, dpv = 0.0;
                        for (int d = 0; d < D; ++d) {
                            dot += (double)qi[d] * (double)kj[d];
                            dpv += (double)doi[d] * (double)vj[d];
                        }
                        double p = exp(scale * dot - lse[(size_t)bh * S + i]);
                        double ds = p * (dpv - delta[(size_t)bh * S + i]);
                        for (int d = 0; d < D; ++d) {
                            ak[d] += ds * (double)qi[d];
                            av[d] += p * (double)doi[d];
                        }
                    }
                    if (dk) {
                        double *o = dk + ((size_t)bh * n_cols + n) * D;
                        for (int d = 0; d < D; ++d) o[d] = scale * ak[d];
                    }
                    if (dv) {
                        double *o = dv + ((size_t)bh * n_cols + n) * D;
                        for (int d = 0; d < D; ++d) o[d] = av[d];
                    }
                }
            }
            free(ak); free(av);
        }
    }
    free(lse); free(delta); free(row_slot);
    return failed ? -1 : threads;
}
