// Softmax arithmetic shared by the tensor-core forward kernels: three-input maximum and the
// exponential on the FMA pipes (Algorithm 1's inner loop computes exp2 of the scaled scores; part
// of them run here instead of on the MUFU unit).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#ifndef HB_POLY_MASK
#define HB_POLY_MASK 3   // pair i of every 16 runs its two exponentials on the FMA pipes when (i & MASK) == MASK (3: one pair in four); 0xff = never
#endif
#ifndef HB_POLY_DEG
#define HB_POLY_DEG 3
#endif

namespace hilberta {

__device__ __forceinline__ float max3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// 2^x for a pair of values on the FMA pipes (no MUFU), with packed fp32x2 instructions:
// x = n + f with n = round(x) (adding 1.5 * 2^23 leaves the integer in the low mantissa
// bits), f in [-0.5, 0.5]; 2^f by a cubic (max relative error 7.8e-5, far below bf16
// rounding), 2^n by an exponent add.  Used for a fixed share of the exponentials so that
// the MUFU unit and the FMA pipes split the work.  x is clamped at -126 (result ~0).
template <int DEG = 3>
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));
    const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
    const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
    float2 p;
    if constexpr (DEG == 2) {
        p = __ffma2_rn(f, make_float2(0.23842697f, 0.23842697f), make_float2(0.7034453f, 0.7034453f));
        p = __ffma2_rn(p, f, make_float2(1.00044307f, 1.00044307f));
    } else {
        p = __ffma2_rn(f, make_float2(0.055088773f, 0.055088773f), make_float2(0.24260406f, 0.24260406f));
        p = __ffma2_rn(p, f, make_float2(0.69327623f, 0.69327623f));
        p = __ffma2_rn(p, f, make_float2(0.99992895f, 0.99992895f));
    }
    p.x = __uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23));
    p.y = __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23));
    return p;
}

// One lane of ex2_poly2 with scalar instructions: the same operations in the same order, hence the
// same bits.
template <int DEG = 3>
__device__ __forceinline__ float ex2_poly1(float x) {
    x = fmaxf(x, -126.f);
    const float t = __fadd_rn(x, 12582912.f);
    const float n = __fadd_rn(t, -12582912.f);
    const float f = __fadd_rn(x, -n);
    float p;
    if constexpr (DEG == 2) {
        p = __fmaf_rn(f, 0.23842697f, 0.7034453f);
        p = __fmaf_rn(p, f, 1.00044307f);
    } else {
        p = __fmaf_rn(f, 0.055088773f, 0.24260406f);
        p = __fmaf_rn(p, f, 0.69327623f);
        p = __fmaf_rn(p, f, 0.99992895f);
    }
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

}  // namespace hilberta
