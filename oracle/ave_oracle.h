/*
 * CPU oracle for scaled-dot-product attention forward with log-sum-exp
 * (and, at the end of this header, for the dense matrix product).
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, plain, fp64 statement of what
 * the attention forward pass computes.  It exists so that the tests, the smoke
 * check and the CPU-baseline leg of the benchmark can compare the CUDA library
 * against something written independently of it.  Nothing in the product path
 * may include, link or call it, and it shares no code with the CUDA library.
 *
 * What it computes (paper Section 2, "standard attention mechanism":
 * S = Q K^T, P = softmax_row(S), O = P V), with the three additions the
 * library's contract makes explicit:
 *   - a scalar `scale` multiplying Q K^T before the softmax,
 *   - an additive 0 / -inf mask (causal, aligned to the bottom-right corner:
 *     key j is visible to query i iff j <= i + (Sk - Sq)),
 *   - the natural-log log-sum-exp of every scaled, masked score row.
 * Grouped-query attention follows Fig. 1 of the paper: query head h reads
 * key/value head h / (H / Hkv).
 *
 * Pins (tests/test_oracle_pins.py): brute force in long double without the
 * max-subtraction; softmax rows sum to one; Q = 0 gives prefix means of V and
 * LSE = ln(#visible); one-hot keys select a V row; shift, permutation and
 * split/merge identities; fp64 torch softmax+matmul; hand-derived closed forms.
 *
 * Layouts (all contiguous, row-major, last index fastest):
 *   q   bf16 bit patterns  [B, H,   Sq, D]
 *   k,v bf16 bit patterns  [B, Hkv, Sk, D]
 *   o   double             [B, H,   Sq, D]
 *   lse double             [B, H,   Sq]
 *   p   double             [B, H,   Sq, Sk]   (optional, may be NULL)
 * Return value: 0 on success, 1 on a bad argument (NULL pointer, non-positive
 * size, H not a multiple of Hkv).  All memory is owned by the caller.
 */
#ifndef AVE_ORACLE_H
#define AVE_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Whole-tensor attention forward, definition above.  Rows are independent and
 * are distributed over OpenMP threads.  A row with no visible key gets O = 0
 * and LSE = -inf. */
int ave_oracle_attn_fwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                        double *o, double *lse, double *p,
                        int B, int H, int Hkv, int Sq, int Sk, int D,
                        int causal, float scale);

/* The same definition evaluated only for `n` selected output rows.
 * rows[3*r+0..2] = (b, h, i).  o is [n, D], lse is [n].  Used to check large
 * problems on sampled rows: an output row depends on its own Q row and on the
 * K/V of its key/value head only. */
int ave_oracle_attn_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                         const int64_t *rows, int64_t n,
                         double *o, double *lse,
                         int B, int H, int Hkv, int Sq, int Sk, int D,
                         int causal, float scale);

/* Independent brute force for tiny inputs: literal loops, exp(t_j) with NO
 * max subtraction, long double accumulators, mask applied with an `if`.
 * Only meaningful while |scale * q.k| stays far below the long double
 * overflow threshold. */
int ave_oracle_bruteforce(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                          double *o, double *lse,
                          int B, int H, int Hkv, int Sq, int Sk, int D,
                          int causal, float scale);

/* Matrix product (the paper's GEMM workload, Section 9: square bf16 matrices), plain
 * definition in fp64:  C[i, j] = sum_k A[i, k] * B[j, k].
 *   a bf16 bit patterns [M, K], b bf16 bit patterns [N, K], c double [M, N], all row-major.
 * Pins (tests/test_oracle_pins.py): a hand-computed 2x3 by 3x2 product that a transposed
 * operand breaks, B = identity, all-ones operands (every entry K), bilinearity under
 * exact power-of-two scaling, and numpy's fp64 matmul on ragged sizes.
 * Returns 0, or 1 on a bad argument. */
int ave_oracle_gemm_tn(const uint16_t *a, const uint16_t *b, double *c, int M, int N, int K);

/* The same definition for n selected entries: idx[2*e+0..1] = (i, j), out[e] = C[i, j]. */
int ave_oracle_gemm_tn_entries(const uint16_t *a, const uint16_t *b, const int64_t *idx, int64_t n, double *out,
                               int M, int N, int K);

/* Number of OpenMP threads ave_oracle_attn_fwd / _rows will use. */
int ave_oracle_threads(void);

#ifdef __cplusplus
}
#endif
#endif
