/* CPU oracle, C twin of the attention part.  TEST INFRASTRUCTURE ONLY: used by the tests
 * (as a second, independently written implementation that pins the NumPy oracle) and as
 * the timed CPU baseline of the bench.  Shares nothing with the CUDA sources.
 *
 * What it computes (Sections 2.1-2.3 of the paper): for every query token of each listed
 * query block, softmax attention over the tokens of the K/V blocks that the block's mask
 * row selects.  Plain two-pass softmax per query token, all arithmetic in double:
 *   s_k = scale * <q, k>;  m = max s_k;  O = sum exp(s_k - m) v_k / sum exp(s_k - m);
 *   LSE = m + log sum exp(s_k - m).
 * Inputs are bf16 bit patterns (the high half of an IEEE float), widened exactly.
 * A task that selects no block gives O = 0 and LSE = -inf.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC oracle_attn.c -o liboracle_attn.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b) {
    uint32_t w = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int oracle_attn_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Q, K, V: one head, row-major [tokens][head_dim] bf16 bit patterns.
 * task_q_block[t]: query block index of task t; its K/V block list is
 * kv_idx[kv_ptr[t] .. kv_ptr[t+1]).  out: [n_tasks][block_q][head_dim] doubles,
 * lse: [n_tasks][block_q] doubles; query tokens >= seq_q are left untouched. */
void oracle_attn_tasks(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                       int head_dim, int block_q, int block_kv, int seq_q, int seq_kv,
                       double scale, int n_tasks, const int32_t *task_q_block,
                       const int32_t *kv_ptr, const int32_t *kv_idx,
                       double *out, double *lse) {
    long total = (long)n_tasks * block_q;
#pragma omp parallel
    {
        double *q = (double *)malloc(sizeof(double) * head_dim);
        double *acc = (double *)malloc(sizeof(double) * head_dim);
#pragma omp for schedule(dynamic, 4)
        for (long w = 0; w < total; ++w) {
            int t = (int)(w / block_q), r = (int)(w % block_q);
            long tok = (long)task_q_block[t] * block_q + r;
            if (tok >= seq_q) continue;
            for (int d = 0; d < head_dim; ++d) q[d] = bf16_to_double(Q[tok * head_dim + d]);
            /* pass 1: maximum score */
            double m = -INFINITY;
            for (int e = kv_ptr[t]; e < kv_ptr[t + 1]; ++e) {
                long k0 = (long)kv_idx[e] * block_kv, k1 = k0 + block_kv;
                if (k1 > seq_kv) k1 = seq_kv;
                for (long k = k0; k < k1; ++k) {
                    double s = 0.0;
                    for (int d = 0; d < head_dim; ++d) s += q[d] * bf16_to_double(K[k * head_dim + d]);
                    s *= scale;
                    if (s > m) m = s;
                }
            }
            double *o = out + w * head_dim;
            if (m == -INFINITY) {
                for (int d = 0; d < head_dim; ++d) o[d] = 0.0;
                lse[w] = -INFINITY;
                continue;
            }
            /* pass 2: normaliser and weighted values */
            double l = 0.0;
            for (int d = 0; d < head_dim; ++d) acc[d] = 0.0;
            for (int e = kv_ptr[t]; e < kv_ptr[t + 1]; ++e) {
                long k0 = (long)kv_idx[e] * block_kv, k1 = k0 + block_kv;
                if (k1 > seq_kv) k1 = seq_kv;
                for (long k = k0; k < k1; ++k) {
                    double s = 0.0;
                    for (int d = 0; d < head_dim; ++d) s += q[d] * bf16_to_double(K[k * head_dim + d]);
                    double p = exp(s * scale - m);
                    l += p;
                    for (int d = 0; d < head_dim; ++d) acc[d] += p * bf16_to_double(V[k * head_dim + d]);
                }
            }
            for (int d = 0; d < head_dim; ++d) o[d] = acc[d] / l;
            lse[w] = m + log(l);
        }
        free(q);
        free(acc);
    }
}
