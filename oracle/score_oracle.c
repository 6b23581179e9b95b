/*
 * TEST INFRASTRUCTURE - float64 CPU oracle for the attention-importance scores.
 *
 * Not part of the product: only tests, the smoke check and the CPU-baseline leg
 * of the benchmark may build or call this file.  It shares no code with the
 * CUDA library.
 *
 * What it computes (Algorithm 1 of the KVCrush paper, first two steps):
 *   A_h = softmax(Q_h K_h^T / sqrt(d_k))            (one S x S matrix per head)
 *   c_h(t) = sum over queries j of A_h(j, t)        (attention received by key t)
 * Algorithm 1 prints the sum with the two indices of A_h swapped, which would be
 * a softmax row sum and therefore identically 1; the column sum is the reading
 * used here (it is also H2O's "sum of attention weights" named in Sec. 2.3).
 * The 1/S normalisation of Algorithm 1 is applied by the caller when wanted.
 *
 * The code is the definition written out: one query row at a time, all logits
 * of the row, the row maximum, the exponentials, their sum, the division, and
 * the accumulation into the column sums.  No tiling, no online softmax.
 * Heads are independent and are spread over OpenMP threads; within a head the
 * rows are visited in order, so the result does not depend on the thread count.
 */
#include <math.h>
#include <stdlib.h>
#include <stddef.h>

/*
 * Q      [L][Hq][D]   float64 (widened storage values), token-major
 * K      [L][Hkv][D]  float64; query head h reads key head h / (Hq/Hkv)
 * causal != 0: query j attends keys t <= j; otherwise all keys
 * colsum [Hq][L] out: c_h(t)
 * lse    [Hq][L] out (may be NULL): log sum_t exp(s(j,t)) for every query j
 * j_begin, j_end: only the query rows j_begin <= j < j_end are visited (0, L = all of them).
 *        With a partial range colsum holds the sum over those rows only - which is the complete
 *        c_h(t) for every key t >= j_begin of a causal sequence (earlier queries do not see t) -
 *        and lse is written for those rows only.  Used to check samples of long sequences.
 * returns 0, or -1 on bad arguments / allocation failure
 */
int kvcrush_oracle_scores(const double *Q, const double *K, int L, int Hq, int Hkv, int D,
                          int causal, double scale, int j_begin, int j_end, double *colsum, double *lse)
{
    if (L < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (j_begin < 0 || j_end > L || j_begin > j_end) return -1;
    const int G = Hq / Hkv;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < Hq; ++h) {
        double *c = colsum + (size_t)h * (size_t)L;
        for (int t = 0; t < L; ++t) c[t] = 0.0;
        double *s = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
        if (!s) {
#pragma omp atomic write
            failed = 1;
            continue;
        }
        const int hk = h / G;
        for (int j = j_begin; j < j_end; ++j) {
            const double *q = Q + ((size_t)j * Hq + h) * D;
            const int n = causal ? j + 1 : L;
            double m = -INFINITY;
            for (int t = 0; t < n; ++t) {
                const double *k = K + ((size_t)t * Hkv + hk) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += q[d] * k[d];
                s[t] = scale * dot;
                if (s[t] > m) m = s[t];
            }
            double z = 0.0;
            for (int t = 0; t < n; ++t) {
                s[t] = exp(s[t] - m);
                z += s[t];
            }
            for (int t = 0; t < n; ++t) c[t] += s[t] / z;
            if (lse) lse[(size_t)h * (size_t)L + j] = m + log(z);
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/* Number of OpenMP threads the scores routine will use (reported by the benchmark). */
#ifdef _OPENMP
#include <omp.h>
int kvcrush_oracle_threads(void) { return omp_get_max_threads(); }
#else
int kvcrush_oracle_threads(void) { return 1; }
#endif
