/*
 * ave_moe -- block-quantised FP8 fused mixture-of-experts layer for NVIDIA B200
 * (sm_100a), C ABI.  Part of libave_attn.so.
 *
 * Operation (the paper's third evaluated kernel family, Section 9: "Fused MoE
 * uses DeepSeek-V3.2's block-quantized FP8 configuration: model dimension 7168,
 * intermediate dimension 2048, top-k 4, 32 experts per GPU"; a correct kernel
 * "must preserve blockwise quantization, route tokens through sorted expert
 * maps" and "quantize up-projection intermediates to FP8").  The paper prints
 * no format; the one taken is the published recipe it cites:
 *   - E4M3 codes ("fn": bias 7, no infinities, largest value 448);
 *   - activations: one fp32 scale per (token, 128 consecutive channels);
 *   - weights: one fp32 scale per block of 128 output rows x 128 input channels;
 *   - for token t and each of its K routed experts e = ids[t,k] with weight w[t,k]:
 *       gate_j = sum_c x[t,c] W13[e, j, c],  up_j = sum_c x[t,c] W13[e, F + j, c]
 *       a_j = silu(gate_j) * up_j,  silu(z) = z / (1 + exp(-z))            (fp32)
 *       a is requantised per 128 columns: s = max|a| / 448, code = E4M3(a / s),
 *       round to nearest even, saturating
 *       y[t, i] += w[t,k] * sum_j a~_j W2[e, i, j]
 *     with x, W13, W2, a~ the dequantised values; y is rounded to bf16 once.
 *   Expert numbers are local to this GPU: a pair whose id is outside [0, E)
 *   belongs to another rank and contributes nothing here.
 *
 * Arithmetic: E4M3 products with fp32 accumulation on the tensor cores inside a
 * scale block, fp32 accumulation across blocks, fp32 activation, bf16 result.
 *
 * All pointers are DEVICE pointers to contiguous arrays (last index fastest):
 *   xq   u8  [T, C]       read      sx   f32 [T, C/128]              read
 *   w13q u8  [E, 2F, C]   read      s13  f32 [E, 2F/128, C/128]      read
 *   w2q  u8  [E, C, F]    read      s2   f32 [E, C/128, F/128]       read
 *   ids  i32 [T, K]       read      wts  f32 [T, K]                  read
 *   y    bf16 [T, C]      written
 * Limits: C and F multiples of 128; T * K < 2^24; E <= 1024.  xq, w13q, w2q and
 * y must be 16-byte aligned.  workspace: DEVICE scratch of at least
 * ave_moe_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller,
 * reusable by later calls on the same stream; it holds the sorted copies of
 * the activations, the intermediates and the routing tables.  Seven kernels are
 * enqueued on `stream`; the call does not synchronise.  Inputs are not written.
 * Errors as for ave_attn_fwd (AVE_ERR_NULL_POINTER, AVE_ERR_BAD_SHAPE,
 * AVE_ERR_MISALIGNED, AVE_ERR_WORKSPACE, AVE_ERR_UNSUPPORTED_DEVICE,
 * AVE_ERR_CUDA), validated before any CUDA call; nothing is launched on error.
 * The sticky device-side time-out status of ave_attn.h applies to these kernels too.
 */
#ifndef AVE_MOE_H
#define AVE_MOE_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

int ave_moe_fused_fwd(const void *xq, const float *sx, const void *w13q, const float *s13,
                      const void *w2q, const float *s2, const int *ids, const float *wts, void *y,
                      int T, int C, int F, int E, int K,
                      void *workspace, size_t workspace_bytes, void *stream);

/* Bytes of device workspace ave_moe_fused_fwd needs; 0 if an argument is invalid. */
size_t ave_moe_workspace_bytes(int T, int C, int F, int E, int K);

#ifdef __cplusplus
}
#endif
#endif
