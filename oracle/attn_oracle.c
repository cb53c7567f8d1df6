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
