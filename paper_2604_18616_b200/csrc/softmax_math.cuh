// Arithmetic helpers of the online softmax: packed fp32x2 operations, 3-input
// maximum, and exp2 evaluated on the FMA pipe so that the exponential unit is
// not the only place probabilities can be computed.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "ptx_sm100.cuh"

namespace ave {

// Returns x through an empty asm statement, so that the compiler knows nothing about the value.  Used
// for the trip count (0 or 1) of a loop around code that only a few steps need: as a plain `if`, the
// compiler predicates such a block into every step; as a second instantiation of the step, the copy is
// tens of KB of instructions that are cold in the instruction cache whenever a tile reaches them.
__device__ __forceinline__ int opaque(int x) {
    asm volatile("" : "+r"(x));
    return x;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// (a.x + b.x, a.y + b.y), both rounded toward -infinity.
__device__ __forceinline__ float2 add2_round_down(float2 a, float2 b) {
    float2 r;
    asm("{\n"
        ".reg .b64 ra, rb, rc;\n"
        "mov.b64 ra, {%2, %3};\n"
        "mov.b64 rb, {%4, %5};\n"
        "add.rm.f32x2 rc, ra, rb;\n"
        "mov.b64 {%0, %1}, rc;\n"
        "}\n"
        : "=f"(r.x), "=f"(r.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return r;
}

// 2^x for two values without the exponential unit.  x = n + f with n = floor(x)
// taken from the mantissa of x + 1.5*2^23 (rounded down), 2^f from a cubic
// fitted on [0, 1) (relative error < 9e-5, far below bf16 resolution), and
// 2^n applied by adding n to the exponent field.  Inputs are clamped to
// >= -127: there n = -127 and f = 0, the cubic gives exactly 1.0 and the
// exponent field becomes 0, so every input <= -127, a masked score's -inf
// included, yields exactly 0 (a row without visible keys must sum to 0).
// Inputs must stay below 2^22 - well above anything a probability relative
// to a (possibly stale) row maximum can reach.
__device__ __forceinline__ float2 exp2_fma_pipe(float2 x) {
    const float kMagic = 12582912.f;  // 1.5 * 2^23
    x.x = fmaxf(x.x, -127.f);
    x.y = fmaxf(x.y, -127.f);
    const float2 t = add2_round_down(x, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
    float2 p = __ffma2_rn(f, make_float2(0.07706618f, 0.07706618f), make_float2(0.22764593f, 0.22764593f));
    p = __ffma2_rn(p, f, make_float2(0.69511658f, 0.69511658f));
    p = __ffma2_rn(p, f, make_float2(1.f, 1.f));
    float2 r;
    r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
    r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
    return r;
}

}  // namespace ave
