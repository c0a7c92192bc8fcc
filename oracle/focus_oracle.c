/*
 * Focus oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the Focus inference hot path computes, written from
 * the paper's definitions.  It shares no code, header, table or helper with the CUDA library and
 * must never be called from the product path; only the tests, the smoke check and the bench's
 * CPU-baseline leg use it.
 *
 * Layouts: every tensor is contiguous, x/q/k/v are bf16 bit patterns (uint16) of shape
 * [H, n, D], centroids are fp32 [Hkv, K, D], masks are uint32 [H, n] with bit g set when the token
 * is a member of group g.  Query head h reads KV head h / (Hq / Hkv).
 *
 * What follows which passage of the paper:
 *   focus_oracle_assign     -- Sec. 2 "Learned grouping" (Eq. 1: score of a token against each of
 *                              the K centroids) and Sec. 2 "Efficiency at inference" / Sec. 3.6
 *                              (each token joins its top-k scoring groups).  The score is the
 *                              cosine between the head vector and the centroid (for unit
 *                              centroids it ranks groups exactly as Eq. 1's dot product does).
 *   focus_oracle_attn_rows  -- Sec. 2 (softmax(QK^T/sqrt(d))V restricted to attended pairs, exact
 *                              softmax with no renormalisation) with the hard mask of Appendix D
 *                              (first equation): pair (i,j) is attended iff j <= i and (i-j <= w
 *                              or the two tokens share a group); "share a group" is the top-k
 *                              rule of Sec. 3.6 (membership sets intersect).
 * Parity status: both functions are pinned by the CPU tests (brute force with an explicit dense
 * mask, closed forms, reductions to textbook causal attention, the Appendix D two-set merge, a
 * hand-worked case).  The paper's perplexity/benchmark numbers are "parity unpinned": they need
 * datasets and trained weights that are not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int focus_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Group assignment (Eq. 1 + top-k rule).
 *   x        bf16 [H, n, D]
 *   C        fp32 [Hkv, K, D]; head h uses centroid set h / (H / Hkv)
 *   masks    out  [H, n]   OR of (1 << g) over the t best groups; order = (cosine descending,
 *                          group index ascending), so exact ties go to the lower index
 *   margins  out  [H, n]   cosine of the t-th best minus cosine of the (t+1)-th best (HUGE_VAL
 *                          when t == K); nullable
 * A zero vector has every cosine defined as 0 (so it joins groups 0..t-1).
 * Returns 0, or -1 on bad arguments.
 */
int focus_oracle_assign(const uint16_t* x, int H, int Hkv, int64_t n, int D,
                        const float* C, int K, int t,
                        uint32_t* masks, double* margins) {
    if (!x || !C || !masks || H < 1 || Hkv < 1 || H % Hkv || n < 1 || D < 1 || K < 1 || K > 32 ||
        t < 1 || t > K)
        return -1;
    const int G = H / Hkv;
    /* centroid norms */
    double* cn = (double*)malloc(sizeof(double) * (size_t)Hkv * K);
    for (int a = 0; a < Hkv * K; ++a) {
        double s = 0;
        for (int d = 0; d < D; ++d) s += (double)C[(size_t)a * D + d] * (double)C[(size_t)a * D + d];
        cn[a] = sqrt(s);
    }
#pragma omp parallel for schedule(static)
    for (int64_t hi = 0; hi < (int64_t)H * n; ++hi) {
        const int h = (int)(hi / n);
        const int hk = h / G;
        const uint16_t* xv = x + (size_t)hi * D;
        double cosv[32];
        int order[32];
        double xn = 0;
        for (int d = 0; d < D; ++d) { double a = bf16_to_f64(xv[d]); xn += a * a; }
        xn = sqrt(xn);
        for (int g = 0; g < K; ++g) {
            const float* c = C + ((size_t)hk * K + g) * D;
            double dot = 0;
            for (int d = 0; d < D; ++d) dot += bf16_to_f64(xv[d]) * (double)c[d];
            double den = xn * cn[hk * K + g];
            cosv[g] = den > 0 ? dot / den : 0.0;
            order[g] = g;
        }
        /* insertion sort: cosine descending, index ascending on ties (stable) */
        for (int a = 1; a < K; ++a) {
            int g = order[a], b = a - 1;
            while (b >= 0 && cosv[order[b]] < cosv[g]) { order[b + 1] = order[b]; --b; }
            order[b + 1] = g;
        }
        uint32_t m = 0;
        for (int a = 0; a < t; ++a) m |= (uint32_t)1 << order[a];
        masks[hi] = m;
        if (margins) margins[hi] = (t == K) ? HUGE_VAL : cosv[order[t - 1]] - cosv[order[t]];
    }
    free(cn);
    return 0;
}

/*
 * Attention for a list of query rows, straight from the definition.
 *   For row (h, i):   kept(j)  =  j <= i  and  ( i - j <= w  or  mq[h,i] & mk[h/G, j] != 0 )
 *                     s_j      =  scale * <q_i, k_j>;   if softcap > 0:  s_j = softcap * tanh(s_j / softcap)
 *                     m = max_kept s_j;  Z = sum_kept exp(s_j - m);  lse = m + log Z
 *                     o = sum_kept exp(s_j - m) / Z * v_j
 *   row_h, row_i  the rows to compute (nrows of them)
 *   O    out [nrows, D], lse out [nrows]
 *   psum out [nrows] (nullable)  sum over kept j of the normalised weight -- must be 1
 *   kept out [nrows] (nullable)  number of kept keys of the row
 * Returns 0, or -1 on bad arguments.
 */
int focus_oracle_attn_rows(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                           int Hq, int Hkv, int64_t n, int D,
                           const uint32_t* mq, const uint32_t* mk, int64_t w,
                           double scale, double softcap,
                           int64_t nrows, const int32_t* row_h, const int64_t* row_i,
                           double* O, double* lse, double* psum, int64_t* kept) {
    if (!q || !k || !v || !mq || !mk || !row_h || !row_i || !O || !lse || Hq < 1 || Hkv < 1 ||
        Hq % Hkv || n < 1 || D < 1 || w < 0 || nrows < 0)
        return -1;
    const int G = Hq / Hkv;
    int bad = 0;
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)n);
        double* qd = (double*)malloc(sizeof(double) * (size_t)D);
        double* acc = (double*)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < nrows; ++r) {
            const int h = row_h[r];
            const int64_t i = row_i[r];
            if (h < 0 || h >= Hq || i < 0 || i >= n) { bad = 1; continue; }
            const int hk = h / G;
            const uint32_t mi = mq[(size_t)h * n + i];
            const uint16_t* qv = q + ((size_t)h * n + i) * D;
            for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(qv[d]);
            double m = -HUGE_VAL;
            int64_t cnt = 0;
            for (int64_t j = 0; j <= i; ++j) {
                const int is_kept = (i - j <= w) || ((mi & mk[(size_t)hk * n + j]) != 0);
                if (!is_kept) { s[j] = -HUGE_VAL; continue; }
                const uint16_t* kv = k + ((size_t)hk * n + j) * D;
                double dot = 0;
                for (int d = 0; d < D; ++d) dot += qd[d] * bf16_to_f64(kv[d]);
                double sj = scale * dot;
                if (softcap > 0) sj = softcap * tanh(sj / softcap);
                s[j] = sj;
                if (sj > m) m = sj;
                ++cnt;
            }
            double Z = 0;
            for (int64_t j = 0; j <= i; ++j)
                if (s[j] != -HUGE_VAL) Z += exp(s[j] - m);
            for (int d = 0; d < D; ++d) acc[d] = 0;
            double ps = 0;
            for (int64_t j = 0; j <= i; ++j) {
                if (s[j] == -HUGE_VAL) continue;
                const double p = exp(s[j] - m) / Z;
                ps += p;
                const uint16_t* vv = v + ((size_t)hk * n + j) * D;
                for (int d = 0; d < D; ++d) acc[d] += p * bf16_to_f64(vv[d]);
            }
            for (int d = 0; d < D; ++d) O[(size_t)r * D + d] = acc[d];
            lse[r] = m + log(Z);
            if (psum) psum[r] = ps;
            if (kept) kept[r] = cnt;
        }
        free(s); free(qd); free(acc);
    }
    return bad ? -1 : 0;
}
