/* Block-quantised FP8 fused MoE, plain fp64 definition.  See ave_oracle_moe.h.
 * TEST INFRASTRUCTURE ONLY. */
#include "ave_oracle_moe.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define GROUP 128
#define E4M3_MAX 448.0f

double ave_oracle_e4m3_decode(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;                 /* the only NaN pattern; there are no infinities */
    if (e == 0) v = ldexp((double)m, -9);              /* subnormal: m * 2^-9 */
    else v = ldexp(1.0 + m / 8.0, e - 7);              /* (1 + m/8) * 2^(e-7) */
    return sign ? -v : v;
}

uint8_t ave_oracle_e4m3_encode(float x)
{
    if (isnan(x)) return 0x7f;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs((double)x);
    if (a >= 448.0) return sign | 0x7e;                /* saturate: 0x7e = 448 */
    if (a < ldexp(1.0, -6)) {                          /* subnormal range: multiples of 2^-9 */
        const double n = nearbyint(ldexp(a, 9));       /* round to nearest, ties to even (default mode) */
        return sign | (uint8_t)n;                      /* n == 8 is the smallest normal, code 0x08 */
    }
    int e;
    (void)frexp(a, &e);                                /* a = f * 2^e, f in [0.5, 1) */
    e -= 1;                                            /* a in [2^e, 2^(e+1)) */
    double n = nearbyint(ldexp(a, 3 - e));             /* significand in units of 1/8: 8 .. 16 */
    if (n == 16.0) {
        n = 8.0;
        e += 1;
    }
    if (e > 8 || (e == 8 && n > 14.0)) return sign | 0x7e;   /* rounded past 448 */
    return sign | (uint8_t)(((e + 7) << 3) | ((int)n - 8));
}

int ave_oracle_quant_groups(const float *a, int64_t n_groups, uint8_t *codes, float *scales)
{
    if (!a || !codes || !scales || n_groups < 0) return 1;
    for (int64_t g = 0; g < n_groups; ++g) {
        float amax = 0.0f;
        for (int c = 0; c < GROUP; ++c) amax = fmaxf(amax, fabsf(a[g * GROUP + c]));
        const float s = (amax > 0.0f) ? amax / E4M3_MAX : 1.0f;          /* fp32 division */
        scales[g] = s;
        for (int c = 0; c < GROUP; ++c) codes[g * GROUP + c] = ave_oracle_e4m3_encode(a[g * GROUP + c] / s);
    }
    return 0;
}

static int moe_bad(const void *a, const void *b, const void *c, const void *d, const void *e, const void *f,
                   const void *g, const void *h, const void *y, int T, int C, int F, int E, int K)
{
    if (!a || !b || !c || !d || !e || !f || !g || !h || !y) return 1;
    if (T <= 0 || C <= 0 || F <= 0 || E <= 0 || K <= 0) return 1;
    if (C % GROUP || F % GROUP) return 1;
    return 0;
}

/* One token: y_row[C]; optionally the requantised intermediates of its K experts. */
static int moe_token(const uint8_t *xq, const float *sx, const uint8_t *w13q, const float *s13,
                     const uint8_t *w2q, const float *s2, const int32_t *ids, const float *wts,
                     int t, double *y_row, uint8_t *aq_out, float *sa_out, int C, int F, int E, int K)
{
    const int CG = C / GROUP, FG = F / GROUP;
    double *x = (double *)malloc(sizeof(double) * C);
    float *a = (float *)malloc(sizeof(float) * F);
    uint8_t *aq = (uint8_t *)malloc(F);
    float *sa = (float *)malloc(sizeof(float) * FG);
    double *ad = (double *)malloc(sizeof(double) * F);
    int rc = 0;
    for (int c = 0; c < C; ++c)
        x[c] = ave_oracle_e4m3_decode(xq[(size_t)t * C + c]) * (double)sx[(size_t)t * CG + c / GROUP];
    for (int i = 0; i < C; ++i) y_row[i] = 0.0;
    for (int k = 0; k < K && !rc; ++k) {
        const int e = ids[(size_t)t * K + k];
        if (e < 0 || e >= E) {
            rc = 1;
            break;
        }
        const uint8_t *w13 = w13q + (size_t)e * 2 * F * C;
        const float *sc13 = s13 + (size_t)e * (2 * FG) * CG;
        for (int j = 0; j < F; ++j) {
            double g = 0.0, u = 0.0;
            for (int c = 0; c < C; ++c) {
                g += x[c] * ave_oracle_e4m3_decode(w13[(size_t)j * C + c]) * (double)sc13[(size_t)(j / GROUP) * CG + c / GROUP];
                u += x[c] * ave_oracle_e4m3_decode(w13[(size_t)(F + j) * C + c]) *
                     (double)sc13[(size_t)((F + j) / GROUP) * CG + c / GROUP];
            }
            a[j] = (float)(g / (1.0 + exp(-g)) * u);   /* silu(gate) * up, rounded to fp32 */
        }
        ave_oracle_quant_groups(a, FG, aq, sa);
        if (aq_out) memcpy(aq_out + (size_t)k * F, aq, F);
        if (sa_out) memcpy(sa_out + (size_t)k * FG, sa, sizeof(float) * FG);
        for (int j = 0; j < F; ++j) ad[j] = ave_oracle_e4m3_decode(aq[j]) * (double)sa[j / GROUP];
        const uint8_t *w2 = w2q + (size_t)e * C * F;
        const float *sc2 = s2 + (size_t)e * CG * FG;
        const double w = (double)wts[(size_t)t * K + k];
        for (int i = 0; i < C; ++i) {
            double acc = 0.0;
            for (int j = 0; j < F; ++j)
                acc += ad[j] * ave_oracle_e4m3_decode(w2[(size_t)i * F + j]) * (double)sc2[(size_t)(i / GROUP) * FG + j / GROUP];
            y_row[i] += w * acc;
        }
    }
    free(x);
    free(a);
    free(aq);
    free(sa);
    free(ad);
    return rc;
}

int ave_oracle_moe_fwd(const uint8_t *xq, const float *sx, const uint8_t *w13q, const float *s13,
                       const uint8_t *w2q, const float *s2, const int32_t *ids, const float *wts,
                       double *y, uint8_t *aq, float *sa, int T, int C, int F, int E, int K)
{
    if (moe_bad(xq, sx, w13q, s13, w2q, s2, ids, wts, y, T, C, F, E, K)) return 1;
    int rc = 0;
#pragma omp parallel for schedule(dynamic) reduction(| : rc)
    for (int t = 0; t < T; ++t)
        rc |= moe_token(xq, sx, w13q, s13, w2q, s2, ids, wts, t, y + (size_t)t * C,
                        aq ? aq + (size_t)t * K * F : NULL, sa ? sa + (size_t)t * K * (F / GROUP) : NULL, C, F, E, K);
    return rc;
}

int ave_oracle_moe_rows(const uint8_t *xq, const float *sx, const uint8_t *w13q, const float *s13,
                        const uint8_t *w2q, const float *s2, const int32_t *ids, const float *wts,
                        const int64_t *tok, int64_t n, double *y, int T, int C, int F, int E, int K)
{
    if (moe_bad(xq, sx, w13q, s13, w2q, s2, ids, wts, y, T, C, F, E, K) || !tok || n < 0) return 1;
    int rc = 0;
#pragma omp parallel for schedule(dynamic) reduction(| : rc)
    for (int64_t r = 0; r < n; ++r) {
        if (tok[r] < 0 || tok[r] >= T) {
            rc |= 1;
            continue;
        }
        rc |= moe_token(xq, sx, w13q, s13, w2q, s2, ids, wts, (int)tok[r], y + (size_t)r * C, NULL, NULL, C, F, E, K);
    }
    return rc;
}
