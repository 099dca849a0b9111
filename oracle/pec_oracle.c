/*
 * Test infrastructure, not product code: a plain fp64 CPU oracle for causal
 * softmax attention with log-sum-exp output.  Only tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it; the GPU library never does.
 *
 * What it computes is the definition itself (paper Eq. 3 with the row softmax
 * of Eq. 4, whose sum runs over the keys up to and including the query's own
 * token): for one query row i, one head h and a key set J,
 *
 *     a_j = scale * sum_d q[i,h,d] * k[j,kvh,d]        (kvh = h / (Hq/Hkv))
 *     M   = max_{j in J} a_j
 *     L   = sum_{j in J} exp(a_j - M)
 *     LSE = M + ln L
 *     O_d = (sum_{j in J} exp(a_j - M) * v[j,kvh,d]) / L
 *
 * J is the union of the given half-open key intervals, cut at the query's own
 * position when `causal` is set.  An empty J gives O = 0 and LSE = -inf (the
 * identity element of the partial-attention merge, Section 2.2's online
 * softmax).  No blocking, no running rescale: scores are stored, then reduced.
 * Inputs are float32 (bf16 values widen exactly); all arithmetic is double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int pec_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* q: [n_rows, hq, d]   k, v: [n_keys, hkv, d]   q_pos: [n_rows] position of
 * each query row in its request (keys are indexed by the same positions).
 * iv_lo/iv_hi: n_iv disjoint half-open key intervals inside [0, n_keys).
 * o: [n_rows, hq, d]   lse: [n_rows, hq].  Returns 0, or -1 on bad arguments,
 * -2 when out of memory. */
int pec_oracle_attn_rows(const float *q, const int64_t *q_pos, int64_t n_rows,
                         const float *k, const float *v, int64_t n_keys,
                         int hq, int hkv, int d,
                         const int64_t *iv_lo, const int64_t *iv_hi, int n_iv,
                         int causal, double scale, double *o, double *lse)
{
    if (hq <= 0 || hkv <= 0 || d <= 0 || hq % hkv != 0 || n_rows < 0 || n_keys < 0) return -1;
    for (int t = 0; t < n_iv; ++t)
        if (iv_lo[t] < 0 || iv_hi[t] > n_keys) return -1;
    const int group = hq / hkv;
    int failed = 0;

#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)(n_keys > 0 ? n_keys : 1));
        int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_keys > 0 ? n_keys : 1));
        if (!a || !idx) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            for (int h = 0; h < hq; ++h) {
                if (!a || !idx) continue;
                const int kvh = h / group;
                const float *qr = q + ((size_t)r * hq + h) * d;
                double *orow = o + ((size_t)r * hq + h) * d;
                /* 1. scaled scores of every visible key */
                int64_t n = 0;
                for (int t = 0; t < n_iv; ++t) {
                    for (int64_t j = iv_lo[t]; j < iv_hi[t]; ++j) {
                        if (causal && j > q_pos[r]) continue;
                        const float *kr = k + ((size_t)j * hkv + kvh) * d;
                        double s = 0.0;
                        for (int c = 0; c < d; ++c) s += (double)qr[c] * (double)kr[c];
                        a[n] = s * scale;
                        idx[n] = j;
                        ++n;
                    }
                }
                for (int c = 0; c < d; ++c) orow[c] = 0.0;
                if (n == 0) {
                    lse[(size_t)r * hq + h] = -INFINITY;
                    continue;
                }
                /* 2. row softmax */
                double m = a[0];
                for (int64_t t = 1; t < n; ++t) if (a[t] > m) m = a[t];
                double l = 0.0;
                for (int64_t t = 0; t < n; ++t) l += exp(a[t] - m);
                /* 3. probability-weighted sum of the value rows */
                for (int64_t t = 0; t < n; ++t) {
                    const double p = exp(a[t] - m) / l;
                    const float *vr = v + ((size_t)idx[t] * hkv + kvh) * d;
                    for (int c = 0; c < d; ++c) orow[c] += p * (double)vr[c];
                }
                lse[(size_t)r * hq + h] = m + log(l);
            }
        }
        free(a);
        free(idx);
    }
    return failed ? -2 : 0;
}
