/*
 * TEST INFRASTRUCTURE -- not part of the product.  Plain, slow, fp64 CPU
 * definition of causal grouped-query softmax attention over a packed batch of
 * sequences.  Used only by the tests, the smoke check and the benchmark's
 * cpu_baseline leg; the CUDA library never links or calls it.
 *
 * What it computes (Preliminaries, "Transformer blocks"; Sec. 3.4 "Execution
 * semantics": each block runs on the compacted active sequence, so keys and
 * values exist only for the tokens that are present in the packed buffer):
 *
 *   for every sequence s, query head h, packed row i in [cu[s], cu[s+1]):
 *     kv = h / (Hq / Hkv)
 *     s_ij  = scale * sum_c Q[i,h,c] * K[j,kv,c]        for cu[s] <= j <= i
 *     m_i   = max_j s_ij
 *     l_i   = sum_j exp(s_ij - m_i)
 *     O[i,h,:] = sum_j exp(s_ij - m_i) / l_i * V[j,kv,:]
 *     lse[i,h] = m_i + log(l_i)
 *
 * No tiling, no online softmax, no reordering: the three loops above written
 * out.  Rows to evaluate are given as a list so that large workloads can be
 * checked on a sample.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

int dash_oracle_num_threads(void);

#ifdef _OPENMP
#include <omp.h>
int dash_oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int dash_oracle_num_threads(void) { return 1; }
#endif

/* Q [n,Hq,D], K,V [n,Hkv,D] fp64 row-major; cu int32 [S+1]; rows int64 [n_rows]
 * (packed row indices); O [n_rows,Hq,D]; lse [n_rows,Hq].  Returns 0, or -1 if
 * a row index lies outside every sequence. */
int dash_oracle_attention(const double *Q, const double *K, const double *V,
                          const int32_t *cu, int S, int Hq, int Hkv, int D,
                          double scale, const int64_t *rows, int64_t n_rows,
                          double *O, double *lse)
{
    int G = Hq / Hkv;
    int bad = 0;
    int64_t work = n_rows * (int64_t)Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t w = 0; w < work; ++w) {
        int64_t ri = w / Hq;
        int h = (int)(w % Hq);
        int64_t i = rows[ri];
        int kv = h / G;
        int64_t start = -1;
        for (int s = 0; s < S; ++s)
            if (i >= cu[s] && i < cu[s + 1]) start = cu[s];
        if (start < 0) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        int64_t len = i - start + 1;
        double *sc = (double *)malloc(sizeof(double) * (size_t)len);
        const double *q = Q + (i * Hq + h) * (int64_t)D;
        double m = -INFINITY;
        for (int64_t j = 0; j < len; ++j) {
            const double *k = K + ((start + j) * Hkv + kv) * (int64_t)D;
            double dot = 0.0;
            for (int c = 0; c < D; ++c) dot += q[c] * k[c];
            sc[j] = dot * scale;
            if (sc[j] > m) m = sc[j];
        }
        double l = 0.0;
        for (int64_t j = 0; j < len; ++j) {
            sc[j] = exp(sc[j] - m);
            l += sc[j];
        }
        double *o = O + (ri * Hq + h) * (int64_t)D;
        for (int c = 0; c < D; ++c) o[c] = 0.0;
        for (int64_t j = 0; j < len; ++j) {
            const double *v = V + ((start + j) * Hkv + kv) * (int64_t)D;
            double p = sc[j] / l;
            for (int c = 0; c < D; ++c) o[c] += p * v[c];
        }
        lse[ri * Hq + h] = m + log(l);
        free(sc);
    }
    return bad ? -1 : 0;
}
