/*
 * ave_attn -- flash-attention forward for NVIDIA B200 (sm_100a), C ABI.
 *
 * Operation (paper Section 2: S = Q K^T, P = softmax_row(S), O = P V, tiled
 * with an online softmax so S is never materialised; Fig. 1 for the
 * grouped-query head mapping idx_h / gqa; Section 9 for the causal workload):
 *
 *   for every batch b, query head h, query row i, with g = h / (H / Hkv):
 *     t_j  = scale * sum_d Q[b,h,i,d] * K[b,g,j,d]          j in [0, Sk)
 *     key j is visible iff !causal or j <= i + (Sk - Sq)
 *     LSE[b,h,i] = ln sum_{visible j} exp(t_j)               (natural log)
 *     O[b,h,i,:] = sum_{visible j} exp(t_j - LSE) * V[b,g,j,:]
 *   A row with no visible key gets O = 0 and LSE = -inf.
 *
 * Arithmetic: bf16 operands, fp32 accumulation on the tensor cores, fp32
 * softmax statistics, probabilities rounded to bf16 for the second product,
 * O rounded to bf16 (round to nearest even) once at the end.
 *
 * Every pointer named "device" must be dereferenceable by the current CUDA
 * device; the caller owns all buffers and the stream.  Calls enqueue work on
 * `stream` and return without synchronising; outputs are valid once the stream
 * reaches that point.  Inputs are never written; outputs must not alias inputs.
 * No call falls back to the CPU: without a compute-capability-10.0 device the
 * launch entry points return AVE_ERR_UNSUPPORTED_DEVICE or AVE_ERR_CUDA.
 *
 * Device-side time-outs are sticky.  Every wait inside a kernel is bounded; a
 * wait that runs out records a code in a status word on that device, and from
 * then on EVERY kernel of this library on that device (attention, split-KV,
 * matrix product) returns at once without touching its outputs, while the
 * launch entry points keep returning AVE_OK (they do not synchronise).  The
 * condition ends when ave_attn_device_status() reads the word, which clears
 * it.  A caller that wants to know whether its results are valid calls
 * ave_attn_device_status() after the work of interest (it synchronises the
 * device) and discards the outputs of every launch since the previous call if
 * it reports AVE_ERR_DEVICE_TIMEOUT.
 *
 * A process may use several GPUs: every launch entry point prepares its kernel
 * on the current device the first time it is used there.
 */
#ifndef AVE_ATTN_H
#define AVE_ATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AVE_OK = 0,
    AVE_ERR_NULL_POINTER = 1,       /* q, k, v, o or lse is NULL */
    AVE_ERR_BAD_SHAPE = 2,          /* a size <= 0, H % Hkv != 0, or a size beyond the limits below */
    AVE_ERR_UNSUPPORTED_D = 3,      /* D not a multiple of 8 in [8, 256] (split-KV calls: not 64 or 128) */
    AVE_ERR_MISALIGNED = 4,         /* q, k, v, o not 16-byte aligned, or lse not 4-byte aligned */
    AVE_ERR_BAD_SCALE = 5,          /* scale is NaN or infinite (zero and negative values are allowed) */
    AVE_ERR_UNSUPPORTED_DEVICE = 6, /* the current device is not compute capability 10.x */
    AVE_ERR_CUDA = 7,               /* a CUDA call failed; see ave_attn_last_cuda_error() */
    AVE_ERR_DEVICE_TIMEOUT = 8,     /* a bounded wait inside a kernel gave up (ave_attn_device_status) */
    AVE_ERR_WORKSPACE = 9,          /* workspace NULL, misaligned or too small */
    AVE_ERR_STATIC_SCRATCH = 10,    /* the problem needs more scratch than the library's built-in array holds */
    AVE_ERR_KERNEL_IMAGE = 11       /* the compiled kernel cannot satisfy its own register split (miscompiled build) */
} ave_status_t;

/*
 * Attention forward, definition at the top of this file (paper Section 2 and
 * Fig. 1).  All pointers are DEVICE pointers to contiguous row-major tensors:
 *   q   bf16 [B, H,   Sq, D]   read
 *   k   bf16 [B, Hkv, Sk, D]   read
 *   v   bf16 [B, Hkv, Sk, D]   read
 *   o   bf16 [B, H,   Sq, D]   written
 *   lse fp32 [B, H,   Sq]      written
 * Limits: D a multiple of 8, 8 <= D <= 256 (the kernels compute with D rounded
 * up to 64, 128 or 256: the loads zero-fill the extra columns, the stores clip
 * them, so D = 96 costs what D = 128 costs and D = 192 what D = 256 costs);
 * H % Hkv == 0; Sq, Sk < 2^31 / 2; B * H < 2^31.
 * causal: 0 = every key visible, nonzero = bottom-right aligned causal mask.
 * scale: multiplies Q K^T before the softmax (callers normally pass 1/sqrt(D)).
 * stream: a cudaStream_t; NULL is the legacy default stream.
 * Arguments are validated in the order of ave_status_t before any CUDA call;
 * on any error nothing is launched and the outputs are untouched.
 * Returns an ave_status_t.
 */
int ave_attn_fwd(const void *q, const void *k, const void *v, void *o, float *lse,
                 int B, int H, int Hkv, int Sq, int Sk, int D,
                 int causal, float scale, void *stream);

/*
 * The same operation for tensors that are not contiguous [B, heads, rows, D]
 * arrays: each of q, k, v, o is described by its base DEVICE pointer and three
 * strides, in ELEMENTS (bf16), of its batch, head and row dimensions, in that
 * order; the D elements of a row are contiguous.  Element (b, h, i, d) of q is
 * at q + b*q_strides[0] + h*q_strides[1] + i*q_strides[2] + d, likewise for
 * k, v (heads = Hkv, rows = Sk) and o.  This covers the paper's Fig. 1 layout
 * (sequence, head, d) -- strides {S*H*D, D, H*D} -- and a packed [B, S, 3, H, D]
 * QKV buffer -- base pointers D*H elements apart, strides {3*S*H*D, D, 3*H*D} --
 * without copies.  lse stays a contiguous fp32 [B, H, Sq] array.
 * Every stride must be positive, a multiple of 8 elements (16 bytes) and below
 * 2^38; a row stride must be at least D.  The strides of o must not make two
 * of its rows overlap (not checked).  The stride arrays are HOST pointers, read
 * before the call returns.  Everything else as for ave_attn_fwd; a NULL stride
 * array is AVE_ERR_NULL_POINTER, a non-positive or too large stride
 * AVE_ERR_BAD_SHAPE, a stride that is not a multiple of 8 AVE_ERR_MISALIGNED.
 */
int ave_attn_fwd_strided(const void *q, const void *k, const void *v, void *o, float *lse,
                         int B, int H, int Hkv, int Sq, int Sk, int D,
                         const long long *q_strides, const long long *k_strides,
                         const long long *v_strides, const long long *o_strides,
                         int causal, float scale, void *stream);

/*
 * The same operation for a batch of sequences of different lengths packed
 * without padding ("varlen").  Token-major DEVICE tensors:
 *   q   bf16 [total_q, H,   D]   read       k, v  bf16 [total_k, Hkv, D]   read
 *   o   bf16 [total_q, H,   D]   written    lse   fp32 [H, total_q]        written
 * Sequence b (0 <= b < B) owns query rows [cu_seqlens_q[b], cu_seqlens_q[b+1])
 * and key rows [cu_seqlens_k[b], cu_seqlens_k[b+1]); attention is computed
 * inside each sequence only, with that sequence's own lengths in the causal
 * rule j <= i + (Sk_b - Sq_b).  cu_seqlens_q and cu_seqlens_k are DEVICE arrays
 * of B + 1 non-decreasing int32 values starting at 0 and ending at total_q and
 * total_k; they are read by the kernel, not by the host, so they are not
 * validated: a sequence longer than max_Sq (queries) or max_Sk (keys), or
 * offsets outside [0, total], give undefined results.  Sequences of length 0
 * are allowed; a sequence with queries but no keys gets O = 0, LSE = -inf.
 * max_Sq / max_Sk: upper bounds of the sequences' lengths (they size the launch;
 * tighter is faster), 1 <= max_Sq <= total_q, 1 <= max_Sk <= total_k.
 * D, H, Hkv, causal, scale, stream, validation order and error behaviour as for
 * ave_attn_fwd.
 */
int ave_attn_fwd_varlen(const void *q, const void *k, const void *v, void *o, float *lse,
                        const int *cu_seqlens_q, const int *cu_seqlens_k,
                        int B, int H, int Hkv, int max_Sq, int max_Sk, int total_q, int total_k,
                        int D, int causal, float scale, void *stream);

/*
 * The same operation for tensors that live in HOST memory (same layouts and
 * limits).  The call enqueues, on `stream`: host-to-device copies of q, k, v
 * into `workspace`, the attention kernel, and device-to-host copies of o and
 * lse.  `workspace` is a DEVICE buffer of at least
 * ave_attn_host_workspace_bytes(...) bytes, 256-byte aligned, owned by the
 * caller and reusable across calls on the same stream.  Copies are
 * asynchronous only when the host buffers are page-locked; either way the
 * results are valid after the stream has been synchronised.
 */
int ave_attn_fwd_host(const void *q_host, const void *k_host, const void *v_host,
                      void *o_host, float *lse_host,
                      int B, int H, int Hkv, int Sq, int Sk, int D,
                      int causal, float scale,
                      void *workspace, size_t workspace_bytes, void *stream);

/* Bytes of device workspace ave_attn_fwd_host needs; 0 if the shape is invalid. */
size_t ave_attn_host_workspace_bytes(int B, int H, int Hkv, int Sq, int Sk, int D);

/*
 * Attention forward with the keys cut into `n_splits` ranges (split-KV): every
 * range is processed as its own work tile with its own online softmax, and a
 * second kernel merges the per-range results through their log-sum-exps,
 *   LSE = ln sum_s exp(LSE_s),   O = sum_s exp(LSE_s - LSE) * O_s,
 * which is the same re-association of the softmax sum that the tiling of paper
 * Section 2 relies on, applied across CTAs.  Same tensors, layouts, limits and
 * result as ave_attn_fwd (up to rounding order), except that D must be 64 or
 * 128; meant for few query rows
 * against many keys (decode, chunked prefill), where one work tile per
 * (batch, head, 256 query rows) would leave most SMs idle.
 * n_splits: 1 .. AVE_SPLITKV_MAX_SPLITS; each range is ceil(Sk / n_splits)
 * keys rounded up to a multiple of 128 (trailing ranges may be empty).
 * workspace: DEVICE scratch of at least ave_attn_splitkv_workspace_bytes(...)
 * bytes, 256-byte aligned, owned by the caller; it holds the fp32 partial
 * outputs and log-sum-exps, is fully rewritten by each call, and may be
 * reused by later calls on the same stream.  Two kernels are enqueued.
 */
#define AVE_SPLITKV_MAX_SPLITS 64
int ave_attn_fwd_splitkv(const void *q, const void *k, const void *v, void *o, float *lse,
                         int B, int H, int Hkv, int Sq, int Sk, int D,
                         int causal, float scale, int n_splits,
                         void *workspace, size_t workspace_bytes, void *stream);

/* Bytes of device workspace ave_attn_fwd_splitkv needs; 0 if an argument is invalid. */
size_t ave_attn_splitkv_workspace_bytes(int B, int H, int Sq, int D, int n_splits);

/*
 * A reasonable n_splits for ave_attn_fwd_splitkv on the current device (148
 * SMs assumed when there is none): the largest count with which all work
 * tiles are resident at once (one wave), no range shorter than 256 keys, at
 * most AVE_SPLITKV_MAX_SPLITS.  Host arithmetic only; 0 if an argument is invalid.
 */
int ave_attn_splitkv_default_splits(int B, int H, int Hkv, int Sq, int Sk, int D);

/*
 * Split-KV attention for callers that must not allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for deployment
 * reasons only.)
 *
 * Some hosts of this library cannot hand it a workspace: an inference server
 * that reserved all device memory for its KV cache at start-up, a real-time
 * loop in which a cudaMalloc (which may synchronise the whole device) is not
 * acceptable, or a plug-in whose host application owns the allocator.  For
 * them this variant of ave_attn_fwd_splitkv keeps its scratch (the fp32
 * partial outputs and log-sum-exps of the key ranges) in an array that is
 * part of the library's device image: AVE_SPLITKV_STATIC_SCRATCH_BYTES bytes
 * on every GPU that loads the library, held until the process exits.  The
 * call itself performs no cudaMalloc/cudaFree and calls no allocating
 * routine; inputs and outputs are still the caller's.
 *
 * Same arguments, layouts and result as ave_attn_fwd_splitkv without the
 * workspace.  A problem whose scratch need,
 * ave_attn_splitkv_workspace_bytes(B, H, Sq, D, n_splits), exceeds
 * AVE_SPLITKV_STATIC_SCRATCH_BYTES is rejected with AVE_ERR_STATIC_SCRATCH
 * and nothing is launched (use fewer ranges, or the workspace variant).
 *
 * The first call on each device looks up the array's device address (with
 * that device current) and remembers it; make that first call outside any
 * stream capture.  All calls on a device share the one array: it keeps the
 * previous call's contents, which is harmless because every call rewrites all
 * the partials it later reads (nothing has to start at zero), but two calls
 * that overlap on the GPU (different streams, no dependency) race on it and
 * give wrong results.  Serialise such calls.
 */
#define AVE_SPLITKV_STATIC_SCRATCH_BYTES (8u << 20)
int ave_attn_fwd_splitkv_static(const void *q, const void *k, const void *v, void *o, float *lse,
                                int B, int H, int Hkv, int Sq, int Sk, int D,
                                int causal, float scale, int n_splits, void *stream);

/*
 * Synchronises the current device, then reads and clears the device-side
 * status word that kernels set when one of their bounded waits (on an
 * mbarrier) runs out.  Returns AVE_OK, AVE_ERR_DEVICE_TIMEOUT (with the raw
 * word in *raw_word if it is not NULL), or AVE_ERR_CUDA.  Bits of the raw word:
 * 1 a TMA load, 2 a tensor-core completion, 4 the softmax warps, 8 a ring slot
 * or a tile-scheduler response did not arrive in time; 16 the wait of
 * ave_attn_selftest_wait_timeout.  While the word is non-zero all kernels of the
 * library on this device are no-ops (see "sticky" at the top of this file).
 */
int ave_attn_device_status(unsigned int *raw_word);

/*
 * The library has two attention kernels for the same operation: one whose CTAs
 * process two 128-row sub-tiles of a 256-row work tile in lock-step (shared K/V
 * loads; the default for long sequences and grouped-query heads), and one with
 * a single 128-row sub-tile per CTA and two CTAs per SM (no lock-step at tile
 * boundaries; better for short causal sequences).  which = 0 lets every call
 * choose by problem shape (the default), 1 / 2 force the first / second for all
 * later calls of this process.  Results agree within rounding order.  Returns
 * AVE_OK, or AVE_ERR_BAD_SHAPE for another value.
 */
#define AVE_KERNEL_AUTO 0
#define AVE_KERNEL_TWO_SUBTILES 1
#define AVE_KERNEL_ONE_SUBTILE 2
int ave_attn_select_kernel(int which);

/* Number of kernels this library has launched in this process so far. */
unsigned long long ave_attn_launch_count(void);

/* Static, human-readable text for a status code. */
const char *ave_attn_strerror(int status);

/* Library version, major * 10000 + minor * 100 + patch. */
int ave_attn_version(void);

/* cudaError_t / CUresult of the last failing CUDA call on this thread. */
int ave_attn_last_cuda_error(void);

/*
 * Diagnostics and self-tests.  (The paper has no counterpart to these; they
 * exist so that the failure paths of the library can be exercised without
 * faulting or hanging a GPU.)
 *
 * ave_attn_tensor_map_encodes: number of times the driver's tensor-map encoder
 * has been called by this process.  The library keeps a small per-thread cache
 * of encoded maps keyed by (pointer, shape, strides, box), so a repeated call
 * on the same buffers encodes nothing.
 *
 * ave_attn_selftest_register_split: AVE_OK if a kernel image compiled with
 * `regs_per_thread` registers per thread could satisfy the register split of
 * the attention kernel's warp roles, else AVE_ERR_KERNEL_IMAGE.  The launch
 * entry points apply the same test to the real image (cudaFuncGetAttributes)
 * before a kernel's first launch on a device and refuse to launch on failure:
 * a register request beyond the CTA's allocation would never return.  Host
 * only; needs no GPU.
 *
 * ave_attn_selftest_inject_failures: make the next `count` kernel launches
 * (what = AVE_INJECT_LAUNCH_FAILURE) or tensor-map encodes (what =
 * AVE_INJECT_ENCODE_FAILURE) of this process fail on the host, before
 * anything reaches the GPU: the affected entry point returns AVE_ERR_CUDA,
 * ave_attn_last_cuda_error() holds the injected code, nothing is launched or
 * counted, outputs are untouched.  count = 0 disarms.
 *
 * ave_attn_selftest_wait_timeout: enqueue a one-warp kernel whose only wait,
 * on a barrier nobody arrives on, uses the library's bounded wait with a limit
 * of 2^limit_cycles_log2 SM cycles (10..26).  The wait runs out, the kernel
 * returns normally and bit 16 of the status word is set, after which the
 * sticky no-op behaviour described at the top of this file can be observed and
 * then cleared with ave_attn_device_status().
 */
#define AVE_INJECT_LAUNCH_FAILURE 1
#define AVE_INJECT_ENCODE_FAILURE 2
unsigned long long ave_attn_tensor_map_encodes(void);
int ave_attn_selftest_register_split(int regs_per_thread);
int ave_attn_selftest_inject_failures(int what, int count);
int ave_attn_selftest_wait_timeout(int limit_cycles_log2, void *stream);

#ifdef __cplusplus
}
#endif
#endif
