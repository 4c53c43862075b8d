// C-ABI entry points of the attention-forward library: argument validation,
// TMA tensor-map encoding, kernel selection and launch.  See include/ave_attn.h
// for the contract of every exported function.
#include "../../include/ave_attn.h"
#include "../../include/ave_gemm.h"
#include "../../include/ave_moe.h"

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "attn_fwd_ws.cuh"
#include "attn_fwd_1t.cuh"
#include "gemm_bf16.cuh"
#include "moe_fp8.cuh"

// Scratch of ave_attn_fwd_splitkv_static: part of the device image, so every GPU that loads the
// library holds it until exit.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_splitkv_static_scratch[AVE_SPLITKV_STATIC_SCRATCH_BYTES];

namespace {

thread_local int t_last_cuda_error = 0;
std::atomic<unsigned long long> g_launches{0};

constexpr int kVersion = 100;  // 0.1.0

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so the
// library does not link against libcuda.
EncodeTiledFn encode_fn() {
    static std::atomic<EncodeTiledFn> cached{nullptr};
    EncodeTiledFn f = cached.load(std::memory_order_acquire);
    if (f) return f;
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !sym) {
        t_last_cuda_error = (e != cudaSuccess) ? int(e) : int(cudaErrorSymbolNotFound);
        return nullptr;
    }
    f = reinterpret_cast<EncodeTiledFn>(sym);
    cached.store(f, std::memory_order_release);
    return f;
}

std::atomic<int> g_inject_launch_failures{0};  // test hook: the next launches fail before reaching the GPU
std::atomic<int> g_inject_encode_failures{0};  // test hook: the next tensor-map encodes fail

bool take_injected(std::atomic<int> &counter) {
    int n = counter.load(std::memory_order_relaxed);
    while (n > 0)
        if (counter.compare_exchange_weak(n, n - 1, std::memory_order_relaxed)) return true;
    return false;
}

// Element strides of one tensor's batch, head and row dimensions (the D elements of a row are contiguous).
struct Strides {
    long long batch, head, row;
};
Strides contiguous_strides(int heads, int rows, int D) {
    return Strides{(long long)heads * rows * D, (long long)rows * D, (long long)D};
}

// bf16 tensor [batch, heads, rows, D] with the given strides as a 4-D map {D, rows, heads, batch} with a
// box of 64 columns x box_rows rows, 128-byte swizzle, zero fill outside the tensor.
struct MapKey {
    const void *base;
    int D, rows, heads, batch, box_rows;
    long long s_batch, s_head, s_row;
    bool operator==(const MapKey &o) const {
        return base == o.base && D == o.D && rows == o.rows && heads == o.heads && batch == o.batch &&
               box_rows == o.box_rows && s_batch == o.s_batch && s_head == o.s_head && s_row == o.s_row;
    }
};
// A tensor map is a pure function of its key (the encoder reads no device state), so repeated calls
// on the same buffers, the common case in a serving loop, reuse the encoded 128 bytes.  Per thread (no
// locks), 16 entries searched linearly and replaced in turn: the handful of maps of one call always fit.
struct MapCache {
    static constexpr int kEntries = 16;
    MapKey key[kEntries];
    CUtensorMap map[kEntries];
    bool valid[kEntries] = {};
    int next = 0;
    const CUtensorMap *find(const MapKey &k) const {
        for (int i = 0; i < kEntries; ++i)
            if (valid[i] && key[i] == k) return &map[i];
        return nullptr;
    }
    void insert(const MapKey &k, const CUtensorMap &m) {
        key[next] = k;
        map[next] = m;
        valid[next] = true;
        next = (next + 1) % kEntries;
    }
};
thread_local MapCache t_map_cache;
std::atomic<unsigned long long> g_map_encodes{0};  // encoder calls so far (a cache hit makes none)

bool encode_map(CUtensorMap *map, const void *base, int D, int rows, int heads, int batch, const Strides &st,
                int box_rows) {
    if (take_injected(g_inject_encode_failures)) {
        t_last_cuda_error = int(CUDA_ERROR_INVALID_VALUE);
        return false;
    }
    const MapKey key{base, D, rows, heads, batch, box_rows, st.batch, st.head, st.row};
    if (const CUtensorMap *hit = t_map_cache.find(key)) {
        *map = *hit;
        return true;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t gdim[4] = {cuuint64_t(D), cuuint64_t(rows), cuuint64_t(heads), cuuint64_t(batch)};
    cuuint64_t gstride[3] = {cuuint64_t(st.row) * 2, cuuint64_t(st.head) * 2, cuuint64_t(st.batch) * 2};
    cuuint32_t box[4] = {64, cuuint32_t(box_rows), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    g_map_encodes.fetch_add(1, std::memory_order_relaxed);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = int(r);
        return false;
    }
    t_map_cache.insert(key, *map);
    return true;
}

int validate(const void *q, const void *k, const void *v, const void *o, const void *lse, int B, int H, int Hkv,
             int Sq, int Sk, int D, float scale) {
    if (!q || !k || !v || !o || !lse) return AVE_ERR_NULL_POINTER;
    if (B <= 0 || H <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return AVE_ERR_BAD_SHAPE;
    if (H % Hkv != 0) return AVE_ERR_BAD_SHAPE;
    if (Sq >= (1 << 30) || Sk >= (1 << 30)) return AVE_ERR_BAD_SHAPE;
    if ((long long)B * H >= (1ll << 31)) return AVE_ERR_BAD_SHAPE;
    if (D < 8 || D > 256 || D % 8 != 0) return AVE_ERR_UNSUPPORTED_D;
    const long long n_qblk = (Sq + ave::BM - 1) / ave::BM;
    if (n_qblk * B * H >= (1ll << 31)) return AVE_ERR_BAD_SHAPE;
    return -1;  // shape checks passed; pointer/scale checks follow
}

int validate_ptrs_and_scale(const void *q, const void *k, const void *v, const void *o, const void *lse,
                            float scale) {
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
         reinterpret_cast<uintptr_t>(o)) & 15u)
        return AVE_ERR_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(lse) & 3u) return AVE_ERR_MISALIGNED;
    if (std::isnan(scale) || std::isinf(scale)) return AVE_ERR_BAD_SCALE;
    return AVE_OK;
}

int check_device() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    static std::atomic<int> ok_mask_lo{0};  // devices 0..30 already checked
    if (dev < 31 && (ok_mask_lo.load(std::memory_order_relaxed) >> dev) & 1) return AVE_OK;
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    if (major != 10) return AVE_ERR_UNSUPPORTED_DEVICE;
    if (dev < 31) ok_mask_lo.fetch_or(1 << dev, std::memory_order_relaxed);
    return AVE_OK;
}

// Per kernel instantiation: the devices (by ordinal) on which the kernel has been prepared.  The
// maximum dynamic shared-memory size is an attribute of a function ON ONE DEVICE, so a process that
// drives several GPUs has to set it once per device, not once per process.
struct PerDeviceOnce {
    std::atomic<unsigned long long> done{0};
    bool is_done(int dev) const { return dev >= 0 && dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1ull); }
    void mark(int dev) {
        if (dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
    }
};

// The softmax warps raise their register count with setmaxnreg.inc, which can only draw on what
// the CTA was given at launch (threads x registers per thread as compiled).  A request beyond that
// never returns, so a kernel image compiled with fewer registers than the split assumes must not
// be launched at all.
bool register_split_fits(int regs_per_thread_at_launch) {
    using Cfg = ave::WsCfg<128>;
    return 128 * Cfg::kRegsLight + 256 * Cfg::kRegsSoftmax <= Cfg::kThreads * regs_per_thread_at_launch;
}
bool register_split_fits_one_subtile(int regs_per_thread_at_launch) {
    using Cfg = ave::OneCfg<128>;
    return 128 * Cfg::kRegsLight + 128 * Cfg::kRegsSoftmax <= Cfg::kThreads * regs_per_thread_at_launch;
}

bool register_split_fits_moe_gemm(int regs_per_thread_at_launch) {
    using Cfg = ave::MoeGemmCfg;
    return 128 * Cfg::kRegsLight + 256 * Cfg::kRegsEpilogue <= Cfg::kThreads * regs_per_thread_at_launch;
}

// Which attention kernel ordinary (not split-KV) launches use: 0 = chosen per problem, 1 = always the
// two-sub-tile kernel, 2 = always the single-sub-tile kernel (ave_attn_select_kernel).
std::atomic<int> g_kernel_choice{0};

// check_register_split: 0 = none, 1 = the two-sub-tile kernel's split, 2 = the single-sub-tile kernel's, 3 = the MoE GEMM's
template <class Kernel>
int prepare_kernel(Kernel kern, int smem_bytes, int check_register_split, PerDeviceOnce &once) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess && once.is_done(dev)) return AVE_OK;
    if (e == cudaSuccess && check_register_split) {
        cudaFuncAttributes attr;
        e = cudaFuncGetAttributes(&attr, kern);
        if (e == cudaSuccess && !(check_register_split == 1   ? register_split_fits(attr.numRegs)
                                  : check_register_split == 2 ? register_split_fits_one_subtile(attr.numRegs)
                                                              : register_split_fits_moe_gemm(attr.numRegs)))
            return AVE_ERR_KERNEL_IMAGE;
    }
    // two CTAs of the single-sub-tile kernel share an SM: ask for the largest shared-memory carve-out
    if (e == cudaSuccess && check_register_split == 2)
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    once.mark(dev);
    return AVE_OK;
}

template <int D, bool CAUSAL, bool SPLIT, bool VARLEN = false>
int launch_ws(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const CUtensorMap &to,
              const ave::FwdParams &p, cudaStream_t stream) {
    using Cfg = ave::WsCfg<D>;
    auto kern = ave::attn_fwd_ws_kernel<D, CAUSAL, SPLIT, VARLEN>;
    static PerDeviceOnce once;  // per instantiation
    const int st = prepare_kernel(kern, Cfg::kSmemBytes, 1, once);
    if (st != AVE_OK) return st;
    if (take_injected(g_inject_launch_failures)) {
        t_last_cuda_error = int(cudaErrorLaunchFailure);
        return AVE_ERR_CUDA;
    }
    kern<<<dim3(p.total_blocks), dim3(Cfg::kThreads), Cfg::kSmemBytes, stream>>>(tq, tk, tv, to, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}


template <int D, bool CAUSAL, bool SPLIT, bool VARLEN = false>
int launch_1t(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const ave::FwdParams &p,
              cudaStream_t stream) {
    using Cfg = ave::OneCfg<D>;
    auto kern = ave::attn_fwd_1t_kernel<D, CAUSAL, SPLIT, VARLEN>;
    static PerDeviceOnce once;  // per instantiation
    const int st = prepare_kernel(kern, Cfg::kSmemBytes, 2, once);
    if (st != AVE_OK) return st;
    if (take_injected(g_inject_launch_failures)) {
        t_last_cuda_error = int(cudaErrorLaunchFailure);
        return AVE_ERR_CUDA;
    }
    kern<<<dim3(p.total_blocks), dim3(Cfg::kThreads), Cfg::kSmemBytes, stream>>>(tq, tk, tv, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}

// Whether an ordinary launch runs the single-sub-tile kernel (two CTAs per SM, 128-row tiles) instead of the
// two-sub-tile one.
bool use_one_subtile(int B, int H, int Hkv, int Sq, int Sk, int causal, bool split, bool varlen) {
    const int choice = g_kernel_choice.load(std::memory_order_relaxed);
    if (choice == 1) return false;
    if (choice == 2) return true;
    (void)B; (void)H; (void)Hkv; (void)Sk; (void)causal; (void)split; (void)varlen;
    // At most 128 query rows per problem (decode, one chunk of a chunked prefill; Sq counts the packed rows of a
    // head-packed split launch): the second sub-tile of a 256-row tile would be empty.  The single-sub-tile
    // kernel then keeps two independent K/V streams per SM in flight, which is what an HBM-bound pass needs
    // (measured on decode shapes: 0.63-0.66 -> 0.76-0.90 of the copy bandwidth).  With more rows the shared
    // K/V loads of the two-sub-tile kernel win (measured 6-15 % on the prefill configurations).
    return Sq <= ave::BM;
}

// Encode the tensor maps, fill the kernel parameters and launch.  n_splits == 1 with no partial
// buffers is the ordinary forward; otherwise every work tile covers one range of keys_per_split keys
// and writes fp32 partials.
// Variable-length launch: token-major tensors [rows, heads, D] and the sequences' row ranges.
struct VarlenArgs {
    const int *cu_q, *cu_k;  // device, B + 1 entries
    int total_q, total_k;
};

// `layout` (strides of q, k, v, o in this order) is NULL for contiguous [B, heads, rows, D] tensors; `varlen`
// is NULL unless the launch is a variable-length one (Sq and Sk are then the longest sequences).
int launch_attention(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv, int Sq,
                     int Sk, int D, int causal, float scale, int n_splits, int keys_per_split, float *o_partial,
                     float *lse_partial, int rows_per_head, const Strides *layout, const VarlenArgs *varlen,
                     cudaStream_t s) {
    auto token_major = [&](int heads, int rows) { return Strides{(long long)rows * heads * D, (long long)D, (long long)heads * D}; };
    const int rows_q = varlen ? varlen->total_q : Sq, rows_k = varlen ? varlen->total_k : Sk, n_batch = varlen ? 1 : B;
    const Strides sq = layout ? layout[0] : varlen ? token_major(H, rows_q) : contiguous_strides(H, Sq, D);
    const Strides sk = layout ? layout[1] : varlen ? token_major(Hkv, rows_k) : contiguous_strides(Hkv, Sk, D);
    const Strides sv = layout ? layout[2] : varlen ? token_major(Hkv, rows_k) : contiguous_strides(Hkv, Sk, D);
    const Strides so = layout ? layout[3] : varlen ? token_major(H, rows_q) : contiguous_strides(H, Sq, D);
    const bool split = o_partial != nullptr;
    // a head dimension above 128 leaves no TMEM for a second sub-tile: only the single-sub-tile kernel has it
    const bool one = D > 128 || use_one_subtile(B, H, Hkv, Sq, Sk, causal, split, varlen != nullptr);
    CUtensorMap tq, tk, tv, to;
    if (!encode_map(&tq, q, D, rows_q, H, n_batch, sq, ave::BM)) return AVE_ERR_CUDA;
    if (!one && !encode_map(&to, o, D, rows_q, H, n_batch, so, ave::WsCfg<128>::kOutBoxRows)) return AVE_ERR_CUDA;
    if (!encode_map(&tk, k, D, rows_k, Hkv, n_batch, sk, ave::BN)) return AVE_ERR_CUDA;
    if (!encode_map(&tv, v, D, rows_k, Hkv, n_batch, sv, ave::BN)) return AVE_ERR_CUDA;

    ave::FwdParams p{};
    p.o = o;
    p.lse = lse;
    p.o_stride_b = so.batch;
    p.o_stride_h = so.head;
    p.o_stride_r = so.row;
    p.d_true = D;
    p.cu_q = varlen ? varlen->cu_q : nullptr;
    p.cu_k = varlen ? varlen->cu_k : nullptr;
    p.lse_stride_h = varlen ? varlen->total_q : 0;
    const int Dk = D <= 64 ? 64 : D <= 128 ? 128 : 256;  // the kernel's head dimension: TMA zero-fills the columns beyond D
    if (!ave::plan_work_tiles(p, B, H, Hkv, Sq, Sk, D, causal != 0, split, n_splits, keys_per_split, rows_per_head, one))
        return AVE_ERR_BAD_SHAPE;
    p.o_partial = o_partial;
    p.lse_partial = lse_partial;
    p.scale_log2 = scale * 1.4426950408889634f;

    if (one && Dk == 256) {  // (the split-KV entry points take 64 or 128 only)
        if (varlen)
            return causal ? launch_1t<256, true, false, true>(tq, tk, tv, p, s) : launch_1t<256, false, false, true>(tq, tk, tv, p, s);
        return causal ? launch_1t<256, true, false>(tq, tk, tv, p, s) : launch_1t<256, false, false>(tq, tk, tv, p, s);
    }
    if (one) {
        if (split) {
            if (Dk == 128)
                return causal ? launch_1t<128, true, true>(tq, tk, tv, p, s) : launch_1t<128, false, true>(tq, tk, tv, p, s);
            return causal ? launch_1t<64, true, true>(tq, tk, tv, p, s) : launch_1t<64, false, true>(tq, tk, tv, p, s);
        }
        if (varlen) {
            if (Dk == 128)
                return causal ? launch_1t<128, true, false, true>(tq, tk, tv, p, s)
                              : launch_1t<128, false, false, true>(tq, tk, tv, p, s);
            return causal ? launch_1t<64, true, false, true>(tq, tk, tv, p, s)
                          : launch_1t<64, false, false, true>(tq, tk, tv, p, s);
        }
        if (Dk == 128)
            return causal ? launch_1t<128, true, false>(tq, tk, tv, p, s) : launch_1t<128, false, false>(tq, tk, tv, p, s);
        return causal ? launch_1t<64, true, false>(tq, tk, tv, p, s) : launch_1t<64, false, false>(tq, tk, tv, p, s);
    }
    if (split) {
        if (Dk == 128)
            return causal ? launch_ws<128, true, true>(tq, tk, tv, to, p, s) : launch_ws<128, false, true>(tq, tk, tv, to, p, s);
        return causal ? launch_ws<64, true, true>(tq, tk, tv, to, p, s) : launch_ws<64, false, true>(tq, tk, tv, to, p, s);
    }
    if (varlen) {
        if (Dk == 128)
            return causal ? launch_ws<128, true, false, true>(tq, tk, tv, to, p, s)
                          : launch_ws<128, false, false, true>(tq, tk, tv, to, p, s);
        return causal ? launch_ws<64, true, false, true>(tq, tk, tv, to, p, s)
                      : launch_ws<64, false, false, true>(tq, tk, tv, to, p, s);
    }
    if (Dk == 128)
        return causal ? launch_ws<128, true, false>(tq, tk, tv, to, p, s) : launch_ws<128, false, false>(tq, tk, tv, to, p, s);
    return causal ? launch_ws<64, true, false>(tq, tk, tv, to, p, s) : launch_ws<64, false, false>(tq, tk, tv, to, p, s);
}

// Combine the partial results of the key ranges of every query row:
//   LSE = ln sum_s exp(LSE_s),  O = sum_s exp(LSE_s - LSE) * O_s.
// One thread per (row, 8 output columns).
__global__ void splitkv_merge_kernel(const float *__restrict__ o_partial, const float *__restrict__ lse_partial,
                                     __nv_bfloat16 *__restrict__ o, float *__restrict__ lse, long long rows, int D,
                                     int n_splits) {
    const int chunks = D / 8;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * chunks) return;
    const long long row = idx / chunks;
    const int ch = int(idx - row * chunks);
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, lse_partial[s * rows + row]);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float denom = 0.f;
    if (m != -INFINITY) {
        for (int s = 0; s < n_splits; ++s) {
            const float w = __expf(lse_partial[s * rows + row] - m);
            denom += w;
            const float4 *src = reinterpret_cast<const float4 *>(o_partial + (s * rows + row) * D + ch * 8);
            const float4 a = src[0], b = src[1];
            acc[0] += w * a.x; acc[1] += w * a.y; acc[2] += w * a.z; acc[3] += w * a.w;
            acc[4] += w * b.x; acc[5] += w * b.y; acc[6] += w * b.z; acc[7] += w * b.w;
        }
    }
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    uint4 out;
    out.x = ave::pack_bf16x2(acc[0] * inv, acc[1] * inv);
    out.y = ave::pack_bf16x2(acc[2] * inv, acc[3] * inv);
    out.z = ave::pack_bf16x2(acc[4] * inv, acc[5] * inv);
    out.w = ave::pack_bf16x2(acc[6] * inv, acc[7] * inv);
    reinterpret_cast<uint4 *>(o + row * D)[ch] = out;
    if (ch == 0) lse[row] = (denom > 0.f) ? m + logf(denom) : -INFINITY;
}

// One warp waits, with the library's bounded wait, on an mbarrier that nobody ever arrives on: the
// wait must give up after `limit_cycles`, record its code in the device status word and return.
__global__ void wait_timeout_selftest_kernel(long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ave::mbar_init(ave::smem_u32(&bar), 1);
        ave::fence_mbar_init();
    }
    __syncthreads();
    ave::mbar_wait_bounded(ave::smem_u32(&bar), 0, &abort_flag, ave::STATUS_TIMEOUT_SELFTEST, limit_cycles);
}

int run_splitkv(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv, int Sq,
                int Sk, int D, int causal, float scale, int n_splits, float *o_partial, float *lse_partial,
                cudaStream_t s) {
    const int kps = ave::splitkv_keys_per_split(Sk, n_splits);
    const int G = H / Hkv;
    const bool pack = ave::splitkv_packs_heads(H, Hkv, Sq);  // query heads of a KV head as rows of one problem
    int st = pack ? launch_attention(q, k, v, o, lse, B, Hkv, Hkv, G * Sq, Sk, D, causal, scale, n_splits, kps,
                                     o_partial, lse_partial, Sq, nullptr, nullptr, s)
                  : launch_attention(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, causal, scale, n_splits, kps, o_partial,
                                     lse_partial, 0, nullptr, nullptr, s);
    if (st != AVE_OK) return st;
    const long long rows = (long long)B * H * Sq;
    const long long work = rows * (D / 8);
    const int threads = 256;
    splitkv_merge_kernel<<<unsigned((work + threads - 1) / threads), threads, 0, s>>>(
        o_partial, lse_partial, static_cast<__nv_bfloat16 *>(o), lse, rows, D, n_splits);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}


// C[M, N] = A[M, K] * B[N, K]^T: tensor maps of the three matrices, tile order, persistent launch.
template <int TN, bool B_NMAJOR>
int launch_gemm_tile(const void *a, const void *b, void *c, int M, int N, int K, int sms, cudaStream_t s) {
    using Cfg = ave::GemmCfg<TN>;
    CUtensorMap ta, tb, tc;
    const Strides sa{(long long)M * K, (long long)M * K, (long long)K};
    const Strides sb{(long long)N * K, (long long)N * K, (long long)(B_NMAJOR ? N : K)};
    const Strides sc{(long long)M * N, (long long)M * N, (long long)N};
    if (!encode_map(&ta, a, K, M, 1, 1, sa, Cfg::kTileM)) return AVE_ERR_CUDA;
    if (B_NMAJOR) {  // B [K, N]: rows of N elements, boxes of 64 columns x 64 rows of K
        if (!encode_map(&tb, b, N, K, 1, 1, sb, Cfg::kSliceK)) return AVE_ERR_CUDA;
    } else {         // B [N, K]: rows of K elements, boxes of 64 columns of K x the tile's rows
        if (!encode_map(&tb, b, K, N, 1, 1, sb, Cfg::kTileN)) return AVE_ERR_CUDA;
    }
    if (!encode_map(&tc, c, N, M, 1, 1, sc, Cfg::kOutBoxRows)) return AVE_ERR_CUDA;
    ave::GemmParams p;
    p.M = M;
    p.N = N;
    p.K = K;
    p.tiles_m = (M + Cfg::kTileM - 1) / Cfg::kTileM;
    p.tiles_n = (N + Cfg::kTileN - 1) / Cfg::kTileN;
    // The ~148 tiles in flight at a time should cover a near-square part of C, which minimises the A and B
    // bytes they pull through L2: 16 block rows x 9 block columns of 128 x 256 is 2048 x 2304 elements.
    p.group_m = 16;
    auto kern = ave::gemm_bf16_kernel<TN, B_NMAJOR>;
    static PerDeviceOnce once;  // per instantiation
    const int st = prepare_kernel(kern, Cfg::kSmemBytes, 0, once);
    if (st != AVE_OK) return st;
    cudaError_t e;
    const long long n_tiles = (long long)p.tiles_m * p.tiles_n;
    const unsigned grid = unsigned(n_tiles < sms ? n_tiles : sms);
    kern<<<dim3(grid), dim3(Cfg::kThreads), Cfg::kSmemBytes, s>>>(ta, tb, tc, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}

template <bool B_NMAJOR>
int launch_gemm(const void *a, const void *b, void *c, int M, int N, int K, cudaStream_t s) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || sms <= 0) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    // 128 x 256 tiles for no more than half of the SMs: halve the tile, so that twice as many SMs work and each
    // finishes earlier (measured: n = 1024 gains a third, while at n = 2048, 128 tiles on 148 SMs, the narrow
    // tile's second wave costs a third)
    const long long wide_tiles = (long long)((M + 127) / 128) * ((N + 255) / 256);
    if (2 * wide_tiles <= sms) return launch_gemm_tile<128, B_NMAJOR>(a, b, c, M, N, K, sms, s);
    return launch_gemm_tile<256, B_NMAJOR>(a, b, c, M, N, K, sms, s);
}

// E4M3 codes [d2, rows, inner] (inner contiguous) as a 4-D map with boxes of 128 bytes x box_rows rows, 128-byte
// swizzle, zero fill outside.  (Not cached: two encodes per GEMM of a layer call.)
bool encode_map_u8(CUtensorMap *map, const void *base, long long inner, long long rows, long long d2, int box_rows) {
    if (take_injected(g_inject_encode_failures)) {
        t_last_cuda_error = int(CUDA_ERROR_INVALID_VALUE);
        return false;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t gdim[4] = {cuuint64_t(inner), cuuint64_t(rows), cuuint64_t(d2), 1};
    cuuint64_t gstride[3] = {cuuint64_t(inner), cuuint64_t(inner) * cuuint64_t(rows), cuuint64_t(inner) * cuuint64_t(rows) * cuuint64_t(d2)};
    cuuint32_t box[4] = {128, cuuint32_t(box_rows), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    g_map_encodes.fetch_add(1, std::memory_order_relaxed);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = int(r);
        return false;
    }
    return true;
}

// fp32 matrix [rows, cols] as a 4-D map {cols, rows, 1, 1} with boxes of 32 columns x 32 rows, 128-byte swizzle.
bool encode_map_f32(CUtensorMap *map, const void *base, long long cols, long long rows) {
    if (take_injected(g_inject_encode_failures)) {
        t_last_cuda_error = int(CUDA_ERROR_INVALID_VALUE);
        return false;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t gdim[4] = {cuuint64_t(cols), cuuint64_t(rows), 1, 1};
    cuuint64_t gstride[3] = {cuuint64_t(cols) * 4, cuuint64_t(cols) * cuuint64_t(rows) * 4, cuuint64_t(cols) * cuuint64_t(rows) * 4};
    cuuint32_t box[4] = {32, 32, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void *>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    g_map_encodes.fetch_add(1, std::memory_order_relaxed);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = int(r);
        return false;
    }
    return true;
}

// Scratch of one fused-MoE call, carved out of the caller's workspace (every part 256-byte aligned).
struct MoeWorkspace {
    long long rows_cap;  // rows of the sorted order, padding included: a multiple of 128
    size_t xq_s, sx_s, ho, aq, sa, row_of, pair_of, w_s, expert_off, cursor, tile_expert, bad_id, total;
};
bool moe_layout(MoeWorkspace &w, int T, int C, int F, int E, int K) {
    if (T <= 0 || C <= 0 || F <= 0 || E <= 0 || K <= 0 || C % 128 || F % 128 || E > 1024) return false;
    const long long pairs = (long long)T * K;
    if (pairs >= (1ll << 24)) return false;
    w.rows_cap = 128 * ((pairs + 127) / 128 + E);  // sum over experts of ceil(rows / 128) tiles is at most this many
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = (off + bytes + 255) & ~size_t(255);
        return at;
    };
    const size_t rows = size_t(w.rows_cap);
    w.xq_s = take(rows * C);
    w.sx_s = take(rows * (C / 128) * 4);
    // the up projection's result h [rows, 2F] is dead once the activations are requantised: the down projection's
    // result o [rows, C] takes the same space
    w.ho = take(rows * size_t(2 * F > C ? 2 * F : C) * 4);
    w.aq = take(rows * F);
    w.sa = take(rows * (F / 128) * 4);
    w.row_of = take(size_t(pairs) * 4);
    w.pair_of = take(rows * 4);
    w.w_s = take(rows * 4);
    w.expert_off = take(size_t(E + 1) * 4);
    w.cursor = take(size_t(E) * 4);
    w.tile_expert = take(rows / 128 * 4);
    w.bad_id = take(4);
    w.total = off;
    return true;
}

int launch_moe_gemm(const void *a, long long rows, const float *a_scale, const void *b, const float *b_scale, int E,
                    int N, int K, const int *tile_expert, const float *row_weight, float *out, int sms, cudaStream_t s) {
    using Cfg = ave::MoeGemmCfg;
    CUtensorMap ta, tb, tc;
    if (!encode_map_u8(&ta, a, K, rows, 1, Cfg::kTile)) return AVE_ERR_CUDA;
    if (!encode_map_u8(&tb, b, K, N, E, Cfg::kTileN)) return AVE_ERR_CUDA;
    if (!encode_map_f32(&tc, out, N, rows)) return AVE_ERR_CUDA;
    ave::MoeGemmParams p;
    p.a_scale = a_scale;
    p.b_scale = b_scale;
    p.tile_expert = tile_expert;
    p.row_weight = row_weight;
    p.out = out;
    p.tiles_m = int(rows / 128);
    p.tiles_n = (N + Cfg::kTileN - 1) / Cfg::kTileN;
    p.nblk = N / 128;
    p.kb = K / 128;
    p.N = N;
    static PerDeviceOnce once;
    const int st = prepare_kernel(ave::moe_gemm_fp8_kernel, Cfg::kSmemBytes, 3, once);
    if (st != AVE_OK) return st;
    if (take_injected(g_inject_launch_failures)) {
        t_last_cuda_error = int(cudaErrorLaunchFailure);
        return AVE_ERR_CUDA;
    }
    const long long n_tiles = (long long)p.tiles_m * p.tiles_n;
    const unsigned grid = unsigned(n_tiles < sms ? n_tiles : sms);
    ave::moe_gemm_fp8_kernel<<<dim3(grid), dim3(Cfg::kThreads), Cfg::kSmemBytes, s>>>(ta, tb, tc, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}

// One of the layer's small kernels has been launched: count it or report the launch error.
int after_small_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}

}  // namespace

extern "C" {

size_t ave_moe_workspace_bytes(int T, int C, int F, int E, int K) {
    MoeWorkspace w;
    return moe_layout(w, T, C, F, E, K) ? w.total : 0;
}

int ave_moe_fused_fwd(const void *xq, const float *sx, const void *w13q, const float *s13, const void *w2q,
                      const float *s2, const int *ids, const float *wts, void *y, int T, int C, int F, int E, int K,
                      void *workspace, size_t workspace_bytes, void *stream) {
    if (!xq || !sx || !w13q || !s13 || !w2q || !s2 || !ids || !wts || !y) return AVE_ERR_NULL_POINTER;
    MoeWorkspace w;
    if (!moe_layout(w, T, C, F, E, K)) return AVE_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(xq) | reinterpret_cast<uintptr_t>(w13q) | reinterpret_cast<uintptr_t>(w2q) |
         reinterpret_cast<uintptr_t>(y)) & 15u)
        return AVE_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(sx) | reinterpret_cast<uintptr_t>(s13) | reinterpret_cast<uintptr_t>(s2) |
         reinterpret_cast<uintptr_t>(ids) | reinterpret_cast<uintptr_t>(wts)) & 3u)
        return AVE_ERR_MISALIGNED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < w.total) return AVE_ERR_WORKSPACE;
    int st = check_device();
    if (st != AVE_OK) return st;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || sms <= 0) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *base = static_cast<uint8_t *>(workspace);
    uint8_t *xq_s = base + w.xq_s;
    float *sx_s = reinterpret_cast<float *>(base + w.sx_s);
    float *ho = reinterpret_cast<float *>(base + w.ho);
    uint8_t *aq = base + w.aq;
    float *sa = reinterpret_cast<float *>(base + w.sa);
    int *row_of = reinterpret_cast<int *>(base + w.row_of);
    int *pair_of = reinterpret_cast<int *>(base + w.pair_of);
    float *w_s = reinterpret_cast<float *>(base + w.w_s);
    int *expert_off = reinterpret_cast<int *>(base + w.expert_off);
    int *cursor = reinterpret_cast<int *>(base + w.cursor);
    int *tile_expert = reinterpret_cast<int *>(base + w.tile_expert);
    int *bad_id = reinterpret_cast<int *>(base + w.bad_id);
    const int pairs = T * K;
    const int rows = int(w.rows_cap);

    // 1. sort the (token, k) pairs by expert
    ave::moe_count_kernel<<<1, 1024, size_t(E) * sizeof(int), s>>>(ids, pairs, E, rows, expert_off, cursor, tile_expert,
                                                                  pair_of, bad_id);
    if ((st = after_small_launch()) != AVE_OK) return st;
    ave::moe_scatter_kernel<<<(pairs + 255) / 256, 256, 0, s>>>(ids, pairs, E, expert_off, cursor, row_of, pair_of);
    if ((st = after_small_launch()) != AVE_OK) return st;
    // 2. the tokens' codes and scales in sorted order
    ave::moe_gather_kernel<<<rows, 128, 0, s>>>(static_cast<const uint8_t *>(xq), sx, wts, pair_of, tile_expert, C, K, xq_s,
                                               sx_s, w_s);
    if ((st = after_small_launch()) != AVE_OK) return st;
    // 3. up projection: h = x W13^T
    st = launch_moe_gemm(xq_s, rows, sx_s, w13q, s13, E, 2 * F, C, tile_expert, nullptr, ho, sms, s);
    if (st != AVE_OK) return st;
    // 4. activation and requantisation
    {
        const long long warps = (long long)rows * (F / 128);
        ave::moe_act_quant_kernel<<<unsigned((warps + 7) / 8), 256, 0, s>>>(ho, tile_expert, F, rows, aq, sa);
        if ((st = after_small_launch()) != AVE_OK) return st;
    }
    // 5. down projection, weighted: o = w * (a W2^T)
    st = launch_moe_gemm(aq, rows, sa, w2q, s2, E, C, F, tile_expert, w_s, ho, sms, s);
    if (st != AVE_OK) return st;
    // 6. every token's K rows summed
    {
        const long long n = (long long)T * (C / 4);
        ave::moe_combine_kernel<<<unsigned((n + 255) / 256), 256, 0, s>>>(ho, row_of, T, C, K, static_cast<__nv_bfloat16 *>(y));
        if ((st = after_small_launch()) != AVE_OK) return st;
    }
    return AVE_OK;
}

int ave_attn_fwd(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv, int Sq,
                 int Sk, int D, int causal, float scale, void *stream) {
    int st = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    st = check_device();
    if (st != AVE_OK) return st;
    return launch_attention(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, causal, scale, 1, 0, nullptr, nullptr, 0, nullptr,
                            nullptr, static_cast<cudaStream_t>(stream));
}

int ave_attn_fwd_strided(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv,
                         int Sq, int Sk, int D, const long long *q_strides, const long long *k_strides,
                         const long long *v_strides, const long long *o_strides, int causal, float scale,
                         void *stream) {
    if (!q_strides || !k_strides || !v_strides || !o_strides) return AVE_ERR_NULL_POINTER;
    int st = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    Strides layout[4];
    const long long *in[4] = {q_strides, k_strides, v_strides, o_strides};
    for (int i = 0; i < 4; ++i) {
        layout[i] = Strides{in[i][0], in[i][1], in[i][2]};
        if (layout[i].batch <= 0 || layout[i].head <= 0 || layout[i].row < D) return AVE_ERR_BAD_SHAPE;
        if (layout[i].batch >= (1ll << 38) || layout[i].head >= (1ll << 38) || layout[i].row >= (1ll << 38))
            return AVE_ERR_BAD_SHAPE;  // the tensor map holds byte strides below 2^40
    }
    for (int i = 0; i < 4; ++i)
        if ((layout[i].batch | layout[i].head | layout[i].row) & 7) return AVE_ERR_MISALIGNED;  // 16-byte units
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    st = check_device();
    if (st != AVE_OK) return st;
    return launch_attention(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, causal, scale, 1, 0, nullptr, nullptr, 0, layout,
                            nullptr, static_cast<cudaStream_t>(stream));
}

int ave_attn_fwd_varlen(const void *q, const void *k, const void *v, void *o, float *lse, const int *cu_seqlens_q,
                        const int *cu_seqlens_k, int B, int H, int Hkv, int max_Sq, int max_Sk, int total_q,
                        int total_k, int D, int causal, float scale, void *stream) {
    if (!cu_seqlens_q || !cu_seqlens_k) return AVE_ERR_NULL_POINTER;
    int st = validate(q, k, v, o, lse, B, H, Hkv, max_Sq, max_Sk, D, scale);
    if (st >= 0) return st;
    if (total_q <= 0 || total_k <= 0 || total_q >= (1 << 30) || total_k >= (1 << 30)) return AVE_ERR_BAD_SHAPE;
    if (max_Sq > total_q || max_Sk > total_k) return AVE_ERR_BAD_SHAPE;
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    if ((reinterpret_cast<uintptr_t>(cu_seqlens_q) | reinterpret_cast<uintptr_t>(cu_seqlens_k)) & 3u)
        return AVE_ERR_MISALIGNED;
    st = check_device();
    if (st != AVE_OK) return st;
    const VarlenArgs vl{cu_seqlens_q, cu_seqlens_k, total_q, total_k};
    return launch_attention(q, k, v, o, lse, B, H, Hkv, max_Sq, max_Sk, D, causal, scale, 1, 0, nullptr, nullptr, 0,
                            nullptr, &vl, static_cast<cudaStream_t>(stream));
}

size_t ave_attn_host_workspace_bytes(int B, int H, int Hkv, int Sq, int Sk, int D) {
    if (validate(&B, &B, &B, &B, &B, B, H, Hkv, Sq, Sk, D, 1.f) >= 0) return 0;
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t qb = up(size_t(B) * H * Sq * D * 2);
    const size_t kb = up(size_t(B) * Hkv * Sk * D * 2);
    const size_t lb = up(size_t(B) * H * Sq * 4);
    return qb /*q*/ + 2 * kb /*k, v*/ + qb /*o*/ + lb /*lse*/;
}

int ave_attn_fwd_host(const void *q_host, const void *k_host, const void *v_host, void *o_host, float *lse_host,
                      int B, int H, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *workspace,
                      size_t workspace_bytes, void *stream) {
    int st = validate(q_host, k_host, v_host, o_host, lse_host, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    if (std::isnan(scale) || std::isinf(scale)) return AVE_ERR_BAD_SCALE;
    const size_t need = ave_attn_host_workspace_bytes(B, H, Hkv, Sq, Sk, D);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return AVE_ERR_WORKSPACE;
    st = check_device();
    if (st != AVE_OK) return st;

    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t q_bytes = size_t(B) * H * Sq * D * 2, kv_bytes = size_t(B) * Hkv * Sk * D * 2;
    const size_t lse_bytes = size_t(B) * H * Sq * 4;
    uint8_t *w = static_cast<uint8_t *>(workspace);
    void *dq = w;
    void *dk = w + up(q_bytes);
    void *dv = w + up(q_bytes) + up(kv_bytes);
    void *d_o = w + up(q_bytes) + 2 * up(kv_bytes);
    float *dl = reinterpret_cast<float *>(w + 2 * up(q_bytes) + 2 * up(kv_bytes));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dk, k_host, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dv, v_host, kv_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    st = ave_attn_fwd(dq, dk, dv, d_o, dl, B, H, Hkv, Sq, Sk, D, causal, scale, stream);
    if (st != AVE_OK) return st;
    if ((e = cudaMemcpyAsync(o_host, d_o, q_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(lse_host, dl, lse_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    return AVE_OK;
}

size_t ave_attn_splitkv_workspace_bytes(int B, int H, int Sq, int D, int n_splits) {
    if (B <= 0 || H <= 0 || Sq <= 0 || (D != 64 && D != 128) || n_splits < 1 || n_splits > AVE_SPLITKV_MAX_SPLITS)
        return 0;
    const size_t rows = size_t(B) * H * Sq;
    return size_t(n_splits) * rows * (size_t(D) + 1) * sizeof(float);
}

int ave_attn_splitkv_default_splits(int B, int H, int Hkv, int Sq, int Sk, int D) {
    if (B <= 0 || H <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || H % Hkv != 0 || (D != 64 && D != 128)) return 0;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;  // no device to ask: the count of the part this library is written for
    return ave::splitkv_default_splits(B, H, Hkv, Sq, Sk, sms, AVE_SPLITKV_MAX_SPLITS);
}

int ave_attn_fwd_splitkv(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv,
                         int Sq, int Sk, int D, int causal, float scale, int n_splits, void *workspace,
                         size_t workspace_bytes, void *stream) {
    int st = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    if (D != 64 && D != 128) return AVE_ERR_UNSUPPORTED_D;
    if (n_splits < 1 || n_splits > AVE_SPLITKV_MAX_SPLITS) return AVE_ERR_BAD_SHAPE;
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    const size_t need = ave_attn_splitkv_workspace_bytes(B, H, Sq, D, n_splits);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need)
        return AVE_ERR_WORKSPACE;
    st = check_device();
    if (st != AVE_OK) return st;
    const size_t rows = size_t(B) * H * Sq;
    float *o_partial = static_cast<float *>(workspace);
    float *lse_partial = o_partial + size_t(n_splits) * rows * D;
    return run_splitkv(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, causal, scale, n_splits, o_partial, lse_partial,
                       static_cast<cudaStream_t>(stream));
}

int ave_attn_fwd_splitkv_static(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H,
                                int Hkv, int Sq, int Sk, int D, int causal, float scale, int n_splits,
                                void *stream) {
    int st = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    if (D != 64 && D != 128) return AVE_ERR_UNSUPPORTED_D;
    if (n_splits < 1 || n_splits > AVE_SPLITKV_MAX_SPLITS) return AVE_ERR_BAD_SHAPE;
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    const size_t need = ave_attn_splitkv_workspace_bytes(B, H, Sq, D, n_splits);
    if (need == 0 || need > size_t(AVE_SPLITKV_STATIC_SCRATCH_BYTES)) return AVE_ERR_STATIC_SCRATCH;
    st = check_device();
    if (st != AVE_OK) return st;

    // Device address of the built-in array, looked up once per device with that device current.
    constexpr int kMaxDevices = 64;
    static std::atomic<void *> scratch_of_device[kMaxDevices];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        t_last_cuda_error = int(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        return AVE_ERR_CUDA;
    }
    void *scratch = scratch_of_device[dev].load(std::memory_order_acquire);
    if (!scratch) {
        e = cudaGetSymbolAddress(&scratch, g_splitkv_static_scratch);
        if (e != cudaSuccess || !scratch) {
            t_last_cuda_error = int(e);
            return AVE_ERR_CUDA;
        }
        scratch_of_device[dev].store(scratch, std::memory_order_release);
    }
    const size_t rows = size_t(B) * H * Sq;
    float *o_partial = static_cast<float *>(scratch);
    float *lse_partial = o_partial + size_t(n_splits) * rows * D;
    return run_splitkv(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, causal, scale, n_splits, o_partial, lse_partial,
                       static_cast<cudaStream_t>(stream));
}

int ave_attn_device_status(unsigned int *raw_word) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    unsigned int word = 0, zero = 0;
    e = cudaMemcpyFromSymbol(&word, ave::g_device_status, sizeof(word));
    if (e == cudaSuccess && word != 0) e = cudaMemcpyToSymbol(ave::g_device_status, &zero, sizeof(zero));
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    if (raw_word) *raw_word = word;
    return word ? AVE_ERR_DEVICE_TIMEOUT : AVE_OK;
}

unsigned long long ave_attn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *ave_attn_strerror(int status) {
    switch (status) {
        case AVE_OK: return "ok";
        case AVE_ERR_NULL_POINTER: return "a required pointer is NULL";
        case AVE_ERR_BAD_SHAPE: return "bad shape: sizes must be positive, H a multiple of Hkv, and within limits";
        case AVE_ERR_UNSUPPORTED_D: return "unsupported head dimension (a multiple of 8 up to 256; 64 or 128 for the split-KV calls)";
        case AVE_ERR_MISALIGNED: return "q, k, v, o must be 16-byte aligned and lse 4-byte aligned";
        case AVE_ERR_BAD_SCALE: return "scale is NaN or infinite";
        case AVE_ERR_UNSUPPORTED_DEVICE: return "the current CUDA device is not compute capability 10.x";
        case AVE_ERR_CUDA: return "a CUDA call failed (see ave_attn_last_cuda_error)";
        case AVE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel gave up";
        case AVE_ERR_WORKSPACE: return "workspace is NULL, misaligned or too small";
        case AVE_ERR_STATIC_SCRATCH:
            return "the problem needs more scratch than the built-in array of ave_attn_fwd_splitkv_static holds";
        case AVE_ERR_KERNEL_IMAGE:
            return "the compiled kernel has fewer registers per thread than its warp roles' register split needs";
        default: return "unknown status";
    }
}

int ave_attn_version(void) { return kVersion; }

int ave_attn_select_kernel(int which) {
    if (which < 0 || which > 2) return AVE_ERR_BAD_SHAPE;
    g_kernel_choice.store(which, std::memory_order_relaxed);
    return AVE_OK;
}

unsigned long long ave_attn_tensor_map_encodes(void) { return g_map_encodes.load(std::memory_order_relaxed); }

int ave_attn_selftest_register_split(int regs_per_thread) {
    return register_split_fits(regs_per_thread) ? AVE_OK : AVE_ERR_KERNEL_IMAGE;
}

int ave_attn_selftest_inject_failures(int what, int count) {
    if (count < 0) return AVE_ERR_BAD_SHAPE;
    if (what == AVE_INJECT_LAUNCH_FAILURE) g_inject_launch_failures.store(count, std::memory_order_relaxed);
    else if (what == AVE_INJECT_ENCODE_FAILURE) g_inject_encode_failures.store(count, std::memory_order_relaxed);
    else return AVE_ERR_BAD_SHAPE;
    return AVE_OK;
}

int ave_attn_selftest_wait_timeout(int limit_cycles_log2, void *stream) {
    if (limit_cycles_log2 < 10 || limit_cycles_log2 > 26) return AVE_ERR_BAD_SHAPE;  // 1 us .. a few tens of ms
    int st = check_device();
    if (st != AVE_OK) return st;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(1ll << limit_cycles_log2);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        t_last_cuda_error = int(e);
        return AVE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return AVE_OK;
}

#ifdef AVE_TRACE
// Trace builds only (not part of the public interface): copies the role
// timeline of the traced CTA, TRACE_ROLES x TRACE_ITERS x TRACE_SLOTS clocks.
int ave_attn_trace_read(long long *out) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(out, ave::g_trace, sizeof(ave::g_trace));
    return e == cudaSuccess ? AVE_OK : AVE_ERR_CUDA;
}
// The life span of the last launch's CTAs: n_ctas x {first ns, last ns, tiles processed}.
int ave_attn_trace_read_spans(unsigned long long *out, int n_ctas) {
    if (n_ctas > ave::TRACE_CTAS) n_ctas = ave::TRACE_CTAS;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(out, ave::g_cta_span, size_t(n_ctas) * 3 * sizeof(unsigned long long));
    return e == cudaSuccess ? AVE_OK : AVE_ERR_CUDA;
}
int ave_attn_trace_clear_spans() {
    void *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, ave::g_cta_span);
    if (e == cudaSuccess) e = cudaMemset(ptr, 0, sizeof(ave::g_cta_span));
    return e == cudaSuccess ? AVE_OK : AVE_ERR_CUDA;
}
#endif

static int gemm_validate(const void *a, const void *b, const void *c, int M, int N, int K) {
    if (!a || !b || !c) return AVE_ERR_NULL_POINTER;
    if (M <= 0 || N <= 0 || K <= 0) return AVE_ERR_BAD_SHAPE;
    const long long lim = 1ll << 39;  // elements: a tensor map holds byte strides below 2^40
    if ((long long)M * K >= lim || (long long)N * K >= lim || (long long)M * N >= lim) return AVE_ERR_BAD_SHAPE;
    if ((long long)((M + 127) / 128) * ((N + 127) / 128) >= (1ll << 31)) return AVE_ERR_BAD_SHAPE;
    if ((K & 7) || (N & 7)) return AVE_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c)) & 15u)
        return AVE_ERR_MISALIGNED;
    return AVE_OK;
}

int ave_gemm_bf16_tn(const void *a, const void *b, void *c, int M, int N, int K, void *stream) {
    int st = gemm_validate(a, b, c, M, N, K);
    if (st != AVE_OK) return st;
    st = check_device();
    if (st != AVE_OK) return st;
    return launch_gemm<false>(a, b, c, M, N, K, static_cast<cudaStream_t>(stream));
}

int ave_gemm_bf16_nn(const void *a, const void *b, void *c, int M, int N, int K, void *stream) {
    int st = gemm_validate(a, b, c, M, N, K);
    if (st != AVE_OK) return st;
    st = check_device();
    if (st != AVE_OK) return st;
    return launch_gemm<true>(a, b, c, M, N, K, static_cast<cudaStream_t>(stream));
}

int ave_attn_last_cuda_error(void) { return t_last_cuda_error; }

}  // extern "C"
