/*
 * CPU oracle for attention forward (see ave_oracle.h).  TEST INFRASTRUCTURE
 * ONLY: plain fp64, no blocking, no fusion, no reordering beyond the
 * definition.  Shares no code with the CUDA library.
 */
#include "ave_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* A bf16 value is the upper 16 bits of an IEEE-754 binary32; widening it to
 * binary64 is exact. */
static double bf16_to_double(uint16_t bits)
{
    uint32_t w = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static int bad_args(const void *q, const void *k, const void *v, const void *o,
                    const void *lse, int B, int H, int Hkv, int Sq, int Sk, int D)
{
    if (!q || !k || !v || !o || !lse) return 1;
    if (B <= 0 || H <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return 1;
    if (H % Hkv != 0) return 1;
    return 0;
}

/*
 * One output row.  Steps, in the order of the definition (paper Section 2):
 *   1. s_j = scale * sum_d Q[i,d] K[j,d]                       (S = Q K^T)
 *   2. explicit additive mask row M_j in {0, -inf}; t_j = s_j + M_j
 *   3. m = max_j t_j ; Z = sum_j exp(t_j - m) ; LSE = m + ln Z
 *      P_j = exp(t_j - m) / Z                                  (row softmax)
 *   4. O[i,d] = sum_j P_j V[j,d]                               (O = P V)
 * t, mask, pr are caller-provided scratch rows of length Sk.
 */
static void attn_row(const uint16_t *qrow, const uint16_t *kh, const uint16_t *vh,
                     int i, int Sq, int Sk, int D, int causal, double scale,
                     double *t, double *mask, double *pr,
                     double *orow, double *lse_out)
{
    for (int j = 0; j < Sk; ++j) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += bf16_to_double(qrow[d]) * bf16_to_double(kh[(size_t)j * D + d]);
        t[j] = scale * acc;
    }
    for (int j = 0; j < Sk; ++j) {
        int visible = !causal || (j <= i + (Sk - Sq));
        mask[j] = visible ? 0.0 : -INFINITY;
    }
    for (int j = 0; j < Sk; ++j) t[j] = t[j] + mask[j];

    double m = -INFINITY;
    for (int j = 0; j < Sk; ++j)
        if (t[j] > m) m = t[j];

    if (m == -INFINITY) { /* no visible key */
        for (int d = 0; d < D; ++d) orow[d] = 0.0;
        for (int j = 0; j < Sk; ++j) pr[j] = 0.0;
        *lse_out = -INFINITY;
        return;
    }
    double Z = 0.0;
    for (int j = 0; j < Sk; ++j) {
        pr[j] = exp(t[j] - m);
        Z += pr[j];
    }
    *lse_out = m + log(Z);
    for (int j = 0; j < Sk; ++j) pr[j] = pr[j] / Z;

    for (int d = 0; d < D; ++d) {
        double acc = 0.0;
        for (int j = 0; j < Sk; ++j)
            acc += pr[j] * bf16_to_double(vh[(size_t)j * D + d]);
        orow[d] = acc;
    }
}

int ave_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int ave_oracle_attn_fwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                        double *o, double *lse, double *p,
                        int B, int H, int Hkv, int Sq, int Sk, int D,
                        int causal, float scale)
{
    if (bad_args(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D)) return 1;
    const int G = H / Hkv; /* query heads per key/value head (Fig. 1: idx_h / gqa) */
    const int64_t nrows = (int64_t)B * H * Sq;
    int failed = 0;

#pragma omp parallel
    {
        double *t = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *mask = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *pr = (double *)malloc(sizeof(double) * (size_t)Sk);
        if (!t || !mask || !pr) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 16)
            for (int64_t r = 0; r < nrows; ++r) {
                int i = (int)(r % Sq);
                int h = (int)((r / Sq) % H);
                int b = (int)(r / ((int64_t)Sq * H));
                int g = h / G;
                const uint16_t *qrow = q + (((size_t)b * H + h) * Sq + i) * D;
                const uint16_t *kh = k + ((size_t)b * Hkv + g) * (size_t)Sk * D;
                const uint16_t *vh = v + ((size_t)b * Hkv + g) * (size_t)Sk * D;
                attn_row(qrow, kh, vh, i, Sq, Sk, D, causal, (double)scale,
                         t, mask, pr, o + (size_t)r * D, lse + r);
                if (p) memcpy(p + (size_t)r * Sk, pr, sizeof(double) * (size_t)Sk);
            }
        }
        free(t);
        free(mask);
        free(pr);
    }
    return failed;
}

int ave_oracle_attn_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                         const int64_t *rows, int64_t n,
                         double *o, double *lse,
                         int B, int H, int Hkv, int Sq, int Sk, int D,
                         int causal, float scale)
{
    if (bad_args(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D)) return 1;
    if (!rows || n < 0) return 1;
    for (int64_t r = 0; r < n; ++r) {
        if (rows[3 * r] < 0 || rows[3 * r] >= B) return 1;
        if (rows[3 * r + 1] < 0 || rows[3 * r + 1] >= H) return 1;
        if (rows[3 * r + 2] < 0 || rows[3 * r + 2] >= Sq) return 1;
    }
    const int G = H / Hkv;
    int failed = 0;

#pragma omp parallel
    {
        double *t = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *mask = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *pr = (double *)malloc(sizeof(double) * (size_t)Sk);
        if (!t || !mask || !pr) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (int64_t r = 0; r < n; ++r) {
                int b = (int)rows[3 * r], h = (int)rows[3 * r + 1], i = (int)rows[3 * r + 2];
                int g = h / G;
                const uint16_t *qrow = q + (((size_t)b * H + h) * Sq + i) * D;
                const uint16_t *kh = k + ((size_t)b * Hkv + g) * (size_t)Sk * D;
                const uint16_t *vh = v + ((size_t)b * Hkv + g) * (size_t)Sk * D;
                attn_row(qrow, kh, vh, i, Sq, Sk, D, causal, (double)scale,
                         t, mask, pr, o + (size_t)r * D, lse + r);
            }
        }
        free(t);
        free(mask);
        free(pr);
    }
    return failed;
}

int ave_oracle_bruteforce(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                          double *o, double *lse,
                          int B, int H, int Hkv, int Sq, int Sk, int D,
                          int causal, float scale)
{
    if (bad_args(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D)) return 1;
    const int G = H / Hkv;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int i = 0; i < Sq; ++i) {
                const int g = h / G;
                long double Z = 0.0L;
                for (int j = 0; j < Sk; ++j) {
                    if (causal && j > i + (Sk - Sq)) continue;
                    long double s = 0.0L;
                    for (int d = 0; d < D; ++d)
                        s += (long double)bf16_to_double(q[(((size_t)b * H + h) * Sq + i) * D + d]) *
                             (long double)bf16_to_double(k[(((size_t)b * Hkv + g) * Sk + j) * D + d]);
                    Z += expl((long double)scale * s);
                }
                const size_t ro = ((size_t)b * H + h) * Sq + i;
                lse[ro] = (Z > 0.0L) ? (double)logl(Z) : -INFINITY;
                for (int d = 0; d < D; ++d) {
                    long double acc = 0.0L;
                    for (int j = 0; j < Sk; ++j) {
                        if (causal && j > i + (Sk - Sq)) continue;
                        long double s = 0.0L;
                        for (int e = 0; e < D; ++e)
                            s += (long double)bf16_to_double(q[(((size_t)b * H + h) * Sq + i) * D + e]) *
                                 (long double)bf16_to_double(k[(((size_t)b * Hkv + g) * Sk + j) * D + e]);
                        acc += expl((long double)scale * s) / Z *
                               (long double)bf16_to_double(v[(((size_t)b * Hkv + g) * Sk + j) * D + d]);
                    }
                    o[ro * D + d] = (Z > 0.0L) ? (double)acc : 0.0;
                }
            }
    return 0;
}


/* ------------------------------------------------------------------ GEMM
 * C[i, j] = sum_k A[i, k] * B[j, k], the plain definition of the matrix product
 * the paper's GEMM workload computes (Section 9: square bf16 matrices), with
 * both operands stored with the reduction index contiguous.  fp64 throughout;
 * rows of C are distributed over OpenMP threads. */
int ave_oracle_gemm_tn(const uint16_t *a, const uint16_t *b, double *c, int M, int N, int K) {
    if (!a || !b || !c || M <= 0 || N <= 0 || K <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += bf16_to_double(a[i * K + k]) * bf16_to_double(b[j * K + k]);
            c[i * N + j] = acc;
        }
    }
    return 0;
}

/* The same definition for `n` selected entries: idx[2*e+0..1] = (i, j), out[e] = C[i, j]. */
int ave_oracle_gemm_tn_entries(const uint16_t *a, const uint16_t *b, const int64_t *idx, int64_t n, double *out,
                               int M, int N, int K) {
    if (!a || !b || !idx || !out || M <= 0 || N <= 0 || K <= 0 || n < 0) return 1;
    for (int64_t e = 0; e < n; ++e)
        if (idx[2 * e] < 0 || idx[2 * e] >= M || idx[2 * e + 1] < 0 || idx[2 * e + 1] >= N) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        const int64_t i = idx[2 * e], j = idx[2 * e + 1];
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
            acc += bf16_to_double(a[i * K + k]) * bf16_to_double(b[j * K + k]);
        out[e] = acc;
    }
    return 0;
}
