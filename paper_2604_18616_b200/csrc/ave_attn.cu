// C-ABI entry points of the attention-forward library: argument validation,
// TMA tensor-map encoding, kernel selection and launch.  See include/ave_attn.h
// for the contract of every exported function.
#include "../../include/ave_attn.h"

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "attn_fwd_ws.cuh"

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

// bf16 tensor [n_mat, rows, D] (D contiguous) as a 3-D map with a box of
// 64 columns x box_rows rows, 128-byte swizzle, zero fill outside the tensor.
bool encode_map(CUtensorMap *map, const void *base, int D, int rows, long long n_mat, int box_rows) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t gdim[3] = {cuuint64_t(D), cuuint64_t(rows), cuuint64_t(n_mat)};
    cuuint64_t gstride[2] = {cuuint64_t(D) * 2, cuuint64_t(rows) * cuuint64_t(D) * 2};
    cuuint32_t box[3] = {64, cuuint32_t(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = int(r);
        return false;
    }
    return true;
}

int validate(const void *q, const void *k, const void *v, const void *o, const void *lse, int B, int H, int Hkv,
             int Sq, int Sk, int D, float scale) {
    if (!q || !k || !v || !o || !lse) return AVE_ERR_NULL_POINTER;
    if (B <= 0 || H <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return AVE_ERR_BAD_SHAPE;
    if (H % Hkv != 0) return AVE_ERR_BAD_SHAPE;
    if (Sq >= (1 << 30) || Sk >= (1 << 30)) return AVE_ERR_BAD_SHAPE;
    if ((long long)B * H >= (1ll << 31)) return AVE_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return AVE_ERR_UNSUPPORTED_D;
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

template <int D, bool CAUSAL>
int launch_ws(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const CUtensorMap &to,
              const ave::FwdParams &p, cudaStream_t stream) {
    using Cfg = ave::WsCfg<D>;
    auto kern = ave::attn_fwd_ws_kernel<D, CAUSAL>;
    static std::atomic<bool> configured{false};  // per instantiation
    if (!configured.load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
        if (e != cudaSuccess) {
            t_last_cuda_error = int(e);
            return AVE_ERR_CUDA;
        }
        configured.store(true, std::memory_order_release);
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

}  // namespace

extern "C" {

int ave_attn_fwd(const void *q, const void *k, const void *v, void *o, float *lse, int B, int H, int Hkv, int Sq,
                 int Sk, int D, int causal, float scale, void *stream) {
    int st = validate(q, k, v, o, lse, B, H, Hkv, Sq, Sk, D, scale);
    if (st >= 0) return st;
    st = validate_ptrs_and_scale(q, k, v, o, lse, scale);
    if (st != AVE_OK) return st;
    st = check_device();
    if (st != AVE_OK) return st;

    CUtensorMap tq, tk, tv, to;
    if (!encode_map(&tq, q, D, Sq, (long long)B * H, ave::BM)) return AVE_ERR_CUDA;
    if (!encode_map(&to, o, D, Sq, (long long)B * H, ave::WsCfg<128>::kOutBoxRows)) return AVE_ERR_CUDA;
    if (!encode_map(&tk, k, D, Sk, (long long)B * Hkv, ave::BN)) return AVE_ERR_CUDA;
    if (!encode_map(&tv, v, D, Sk, (long long)B * Hkv, ave::BN)) return AVE_ERR_CUDA;

    ave::FwdParams p;
    p.o = o;
    p.lse = lse;
    p.H = H;
    p.Hkv = Hkv;
    p.Sq = Sq;
    p.Sk = Sk;
    p.BH = B * H;
    p.n_qblk = (Sq + 2 * ave::BM - 1) / (2 * ave::BM);
    p.total_blocks = p.n_qblk * p.BH;
    {
        // Launch (b, h) pairs in groups whose K and V together stay within a slice of L2,
        // whole key/value heads at a time.
        const long long kv_bytes_per_kv_head = 2ll * Sk * D * 2;
        const int G = H / Hkv;
        const long long budget = 64ll << 20;
        long long kv_heads = budget / kv_bytes_per_kv_head;
        if (kv_heads < 1) kv_heads = 1;
        long long hpg = kv_heads * G;
        if (hpg > p.BH) hpg = p.BH;
        p.heads_per_group = int(hpg);
    }
    p.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (D == 128)
        return causal ? launch_ws<128, true>(tq, tk, tv, to, p, s) : launch_ws<128, false>(tq, tk, tv, to, p, s);
    return causal ? launch_ws<64, true>(tq, tk, tv, to, p, s) : launch_ws<64, false>(tq, tk, tv, to, p, s);
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
        case AVE_ERR_UNSUPPORTED_D: return "unsupported head dimension (D must be 64 or 128)";
        case AVE_ERR_MISALIGNED: return "q, k, v, o must be 16-byte aligned and lse 4-byte aligned";
        case AVE_ERR_BAD_SCALE: return "scale is NaN or infinite";
        case AVE_ERR_UNSUPPORTED_DEVICE: return "the current CUDA device is not compute capability 10.x";
        case AVE_ERR_CUDA: return "a CUDA call failed (see ave_attn_last_cuda_error)";
        case AVE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel gave up";
        case AVE_ERR_WORKSPACE: return "workspace is NULL, misaligned or too small";
        default: return "unknown status";
    }
}

int ave_attn_version(void) { return kVersion; }

#ifdef AVE_TRACE
// Trace builds only (not part of the public interface): copies the role
// timeline of the traced CTA, TRACE_ROLES x TRACE_ITERS x TRACE_SLOTS clocks.
int ave_attn_trace_read(long long *out) {
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(out, ave::g_trace, sizeof(ave::g_trace));
    return e == cudaSuccess ? AVE_OK : AVE_ERR_CUDA;
}
#endif

int ave_attn_last_cuda_error(void) { return t_last_cuda_error; }

}  // extern "C"
