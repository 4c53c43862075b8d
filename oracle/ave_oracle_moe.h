/*
 * CPU oracle for the block-quantised FP8 fused mixture-of-experts layer (the
 * paper's third kernel family, Section 9: "DeepSeek-V3.2's block-quantized FP8
 * configuration: model dimension 7168, intermediate dimension 2048, top-k 4,
 * 32 experts per GPU"; "quantize up-projection intermediates to FP8"; "preserve
 * blockwise quantization, route tokens through sorted expert maps").
 *
 * TEST INFRASTRUCTURE ONLY, like ave_oracle.h: plain, slow, fp64; shares no
 * code with the CUDA library; only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may use it.
 *
 * The paper names the configuration but prints no format.  The reading taken
 * (the published DeepSeek-V3 recipe the paper cites):
 *   - FP8 is E4M3 "fn": 1 sign, 4 exponent (bias 7), 3 mantissa bits; no
 *     infinities; 0x7f / 0xff are NaN; largest finite value 448; subnormals
 *     below 2^-6 in steps of 2^-9.
 *   - Activations are quantised per token and per group of 128 consecutive
 *     channels: one fp32 scale s per (token, group), value = code * s.
 *   - Weights are quantised per block of 128 x 128 (output rows x input
 *     channels): one fp32 scale per block.
 *   - Quantising a group of fp32 values a: s = max|a| / 448 computed in fp32
 *     (s = 1 if the group is all zero), code = E4M3(a / s) with the division in
 *     fp32, round to nearest even, saturating at +-448.
 *   - Layer, for token t with its K routed experts e_k = ids[t,k] and routing
 *     weights w[t,k] (ids are local expert numbers in [0, E); tokens of other
 *     ranks' experts are not part of this GPU's problem):
 *         g_j = sum_c x[t,c] * W1[e,j,c]          j in [0, F)   "gate"
 *         u_j = sum_c x[t,c] * W3[e,j,c]                        "up"
 *         a_j = silu(g_j) * u_j,   silu(z) = z / (1 + exp(-z))
 *         a is rounded to fp32 and requantised to FP8 per group of 128 (above)
 *         y_i = sum_k w[t,k] * sum_j a~_j * W2[e_k,i,j]  i in [0, C)
 *     with x, W1, W3, W2, a~ the dequantised values.  W1 and W3 are stored
 *     together as W13[e, 2F, C] (rows [0,F) gate, rows [F,2F) up).
 * Sums are taken in fp64 over exactly dequantised operands; the one place a
 * floating-point value decides an integer, the FP8 code of a, is decided in
 * fp32 as stated, which is also how the CUDA path decides it.
 *
 * Layouts (contiguous, last index fastest):
 *   xq   u8  [T, C]        sx   f32 [T, C/128]
 *   w13q u8  [E, 2F, C]    s13  f32 [E, 2F/128, C/128]
 *   w2q  u8  [E, C, F]     s2   f32 [E, C/128, F/128]
 *   ids  i32 [T, K]        wts  f32 [T, K]
 *   y    f64 [T, C]        (optional) aq u8 [T, K, F], sa f32 [T, K, F/128]
 * C and F are multiples of 128.  Return value: 0, or 1 on a bad argument
 * (NULL pointer, non-positive size, C or F not a multiple of 128, an id
 * outside [0, E)).
 */
#ifndef AVE_ORACLE_MOE_H
#define AVE_ORACLE_MOE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Value of an E4M3 code (NaN for 0x7f and 0xff). */
double ave_oracle_e4m3_decode(uint8_t code);

/* E4M3 code of an fp32 value: round to nearest even, saturate at +-448, NaN -> 0x7f. */
uint8_t ave_oracle_e4m3_encode(float x);

/* Quantise n_groups groups of 128 fp32 values: codes [n_groups*128], scales [n_groups]. */
int ave_oracle_quant_groups(const float *a, int64_t n_groups, uint8_t *codes, float *scales);

/* The layer, definition above.  Rows of y are independent (OpenMP over tokens). */
int ave_oracle_moe_fwd(const uint8_t *xq, const float *sx, const uint8_t *w13q, const float *s13,
                       const uint8_t *w2q, const float *s2, const int32_t *ids, const float *wts,
                       double *y, uint8_t *aq, float *sa, int T, int C, int F, int E, int K);

/* The same for n selected tokens: tok[r] in [0, T); y is [n, C]. */
int ave_oracle_moe_rows(const uint8_t *xq, const float *sx, const uint8_t *w13q, const float *s13,
                        const uint8_t *w2q, const float *s2, const int32_t *ids, const float *wts,
                        const int64_t *tok, int64_t n, double *y, int T, int C, int F, int E, int K);

#ifdef __cplusplus
}
#endif
#endif
