/*
 * ave_gemm -- dense bf16 matrix multiplication for NVIDIA B200 (sm_100a), C ABI.
 *
 * Operation (the paper's first evaluated kernel family, Section 9: a product of
 * square bf16 matrices with normally distributed entries; the paper fixes no
 * memory layout, so both operands are taken with the reduction index
 * contiguous, the form a weight matrix is stored in):
 *
 *   C[i, j] = sum_{k < K} A[i, k] * B[j, k]        i in [0, M), j in [0, N)
 *
 * Arithmetic: bf16 operands, exact products, fp32 accumulation on the tensor
 * cores, C rounded to bf16 (round to nearest even) once at the end.
 *
 * Status codes, error reporting (ave_attn_strerror, ave_attn_last_cuda_error,
 * ave_attn_device_status) and the rules on ownership and asynchrony are those
 * of ave_attn.h: the caller owns all buffers and the stream, the call enqueues
 * on `stream` and returns without synchronising, nothing falls back to the CPU.
 */
#ifndef AVE_GEMM_H
#define AVE_GEMM_H

#include "ave_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * a: bf16 [M, K] row-major, device, read.   b: bf16 [N, K] row-major, device, read.
 * c: bf16 [M, N] row-major, device, written; must not alias a or b.
 * M, N, K > 0; K and N multiples of 8 (rows of 16-byte multiples, a TMA rule);
 * M * K, N * K, M * N below 2^40 elements.  a, b, c 16-byte aligned.
 * Errors, checked in this order before any CUDA call, nothing launched:
 * AVE_ERR_NULL_POINTER, AVE_ERR_BAD_SHAPE (sizes), AVE_ERR_MISALIGNED
 * (K or N not a multiple of 8, or a pointer not 16-byte aligned); then
 * AVE_ERR_UNSUPPORTED_DEVICE / AVE_ERR_CUDA from the launch.
 */
int ave_gemm_bf16_tn(const void *a, const void *b, void *c, int M, int N, int K, void *stream);

/*
 * The same product with B stored the other way round, the plain C = A B of the paper's Section 9 workload:
 *   C[i, j] = sum_{k < K} A[i, k] * B[k, j]
 * a: bf16 [M, K] row-major.  b: bf16 [K, N] row-major.  c: bf16 [M, N] row-major.  Same limits, alignment
 * rules, errors and arithmetic as ave_gemm_bf16_tn; B is read in place (no transposition pass).
 */
int ave_gemm_bf16_nn(const void *a, const void *b, void *c, int M, int N, int K, void *stream);

#ifdef __cplusplus
}
#endif

#endif /* AVE_GEMM_H */
