// Shared definitions of the attention-forward kernels: tile sizes, kernel
// parameters, tcgen05 descriptor encodings, bounded mbarrier waits.
#pragma once

#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "ptx_sm100.cuh"
#include "work_tiles.cuh"

namespace ave {

// Device-side status word; a kernel ORs a code in when a bounded wait gives up.
// (This header is included by exactly one translation unit.)
__device__ unsigned int g_device_status = 0;

constexpr unsigned int STATUS_TIMEOUT_LOAD = 1u;     // waiting for a TMA load
constexpr unsigned int STATUS_TIMEOUT_MMA = 2u;      // waiting for a tcgen05.commit
constexpr unsigned int STATUS_TIMEOUT_SOFTMAX = 4u;  // MMA warp waiting for P
constexpr unsigned int STATUS_TIMEOUT_SLOT = 8u;     // producer waiting for a free stage
constexpr unsigned int STATUS_TIMEOUT_SELFTEST = 16u; // the wait of the time-out self-test (meant to run out)

// A wait is abandoned after this many SM clock cycles (a fraction of a second;
// legitimate waits last microseconds).
constexpr long long WAIT_LIMIT_CYCLES = 1ll << 29;
// Poll limit of the short non-suspending drain loops that run after a wait was abandoned.
constexpr uint32_t WAIT_LIMIT = 1u << 16;

// tcgen05 instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B,
// A K-major (or in TMEM), B K-major (b_mn_major = 0) or MN-major (= 1).
__host__ __device__ constexpr uint32_t make_idesc_bf16(int m, int n, int b_mn_major) {
    return (1u << 4)                         // D format: f32
           | (1u << 7)                       // A format: bf16
           | (1u << 10)                      // B format: bf16
           | (0u << 15)                      // A major: K
           | (uint32_t(b_mn_major) << 16)    // B major
           | (uint32_t(n >> 3) << 17)        // N / 8
           | (uint32_t(m >> 4) << 24);       // M / 16
}

// Shared-memory matrix descriptor, 128-byte swizzle, without the address.
//   K-major operand  (rows of 64 bf16 = 128 B, 8-row atoms of 1024 B):
//       lbo unused (16), sbo = 1024 (next 8 rows)
//   MN-major operand (64 contiguous bf16 along MN per K row of 128 B):
//       lbo = bytes between 64-wide MN groups, sbo = 1024 (next 8 K rows)
__host__ __device__ constexpr uint64_t make_sdesc_sw128(uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16) | (uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32) |
           (1ull << 46)    // descriptor version for sm_100
           | (2ull << 61); // swizzle mode: 128 B
}

// Optional role timeline (builds with -DAVE_TRACE=<cta index> only): SM clock
// stamps of one CTA, [role][iteration][slot], read back by a debug entry point.
#ifdef AVE_TRACE
constexpr int TRACE_ROLES = 4, TRACE_ITERS = 64, TRACE_SLOTS = 8;
__device__ long long g_trace[TRACE_ROLES][TRACE_ITERS][TRACE_SLOTS];
__device__ __forceinline__ void trace_stamp(int role, int iter, int slot) {
    if (blockIdx.x == AVE_TRACE && iter < TRACE_ITERS) g_trace[role][iter][slot] = clock64();
}
// Life span of every CTA of the last launch: global-timer nanoseconds at its first and last instruction
// and the number of work tiles it processed (how long the grid takes to start, how ragged its end is).
constexpr int TRACE_CTAS = 8192;
__device__ unsigned long long g_cta_span[TRACE_CTAS][3];
__device__ __forceinline__ void span_stamp(int slot, unsigned long long value = ~0ull) {
    if (blockIdx.x >= TRACE_CTAS) return;
    if (value == ~0ull) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(value));
    g_cta_span[blockIdx.x][slot] = value;
}
#else
__device__ __forceinline__ void trace_stamp(int, int, int) {}
__device__ __forceinline__ void span_stamp(int, unsigned long long = 0) {}
#endif

// Wait for an mbarrier phase, for a bounded TIME (one mbarrier.try_wait may
// itself suspend the thread for a hardware-chosen while, so counting polls
// does not bound the wait).  Returns false when the time ran out or another
// thread of the CTA has already given up; `abort_flag` is a shared-memory
// word all roles watch.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                                  unsigned int code, long long limit_cycles = WAIT_LIMIT_CYCLES) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag != 0) return false;
        if (clock64() - t0 > limit_cycles) break;
    }
    *abort_flag = 1;
    atomicOr(&g_device_status, code);
    return false;
}

}  // namespace ave
