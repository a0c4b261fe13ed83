// Counter-based Gaussian noise on the device: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)
// and a float32 Box-Muller transform.  The stream definition (key, counter words, tags, uniform
// map, pairing) is the one stated at the top of bgrpo.h.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "internal.h"

namespace bgrpo {

__device__ __forceinline__ void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
    uint64_t p;
    asm("mul.wide.u32 %0, %1, %2;" : "=l"(p) : "r"(a), "r"(b));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p));
}

// Ten rounds; one round sends (c0,c1,c2,c3) to (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0))
// and the key advances by the Weyl constants between rounds (the host has tabulated the ten keys).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const PhiloxKeys& keys) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo(kPhiloxM0, c.x, hi0, lo0);
        mulhilo(kPhiloxM1, c.z, hi1, lo1);
        c = make_uint4(hi1 ^ c.y ^ keys.k[r][0], lo1, hi0 ^ c.w ^ keys.k[r][1], lo0);
    }
    return c;
}

// u = ((x >> 9) + 0.5) * 2^-23, built without an integer-to-float conversion: the 23 kept bits become the
// mantissa of a float in [1, 2), and subtracting 1 - 2^-24 is exact.
__device__ __forceinline__ float uniform_open(uint32_t x) {
    return __uint_as_float((x >> 9) | 0x3f800000u) - 0.99999994f;
}

// Hardware special-function approximations (flush-to-zero forms: one MUFU each, no denormal fix-up code).
__device__ __forceinline__ float fast_sqrt(float x) {
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_sin(float x) {
    float y;
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_cos(float x) {
    float y;
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One Box-Muller pair from two words: (r cos 2 pi u_b, r sin 2 pi u_b), r = sqrt(-2 ln u_a).
//
// Accuracy (the result must stay within ~1e-4 of the exact value so that g * xi, g ~ 0.1, moves a
// latent by well under 1e-5):
//  * -2 ln u_a comes from the hardware log2 (absolute error 2^-22 for arguments in (0.5, 2), relative
//    2^-22 elsewhere).  An absolute error in r^2 becomes a large relative error in r only when r is tiny,
//    i.e. u_a within 2^-9 of 1; there w = 1 - u_a is exact in float32 and the series
//    -2 ln(1 - w) = 2w + w^2 + ... (truncation below 1.3e-6 relative) replaces the log.
//  * the angle is folded to (-pi, pi), where the hardware sine/cosine are good to about 4e-7 absolute,
//    and the sign change is absorbed into r.
__device__ __forceinline__ float2 box_muller(uint32_t wa, uint32_t wb) {
    const float ua = uniform_open(wa);
    const float w = 1.0f - ua;
    const float series = fmaf(w, w, w + w);
    const float viaLog = -1.3862944f * fast_log2(ua);          // -2 ln 2 * log2(u)
    const float r2 = (w < 0.001953125f) ? series : viaLog;
    const float nr = -fast_sqrt(r2);
    // 2 pi u_b - pi with u_b = m - (1 - 2^-24), m in [1, 2) the float built from the word's top 23 bits: the constant
    // term takes the subtraction in (its float32 rounding moves the angle by < 5e-7, i.e. xi by < 3e-6)
    const float th = fmaf(__uint_as_float((wb >> 9) | 0x3f800000u), 6.2831855f, -9.4247776f);
    return make_float2(nr * fast_cos(th), nr * fast_sin(th));
}

__device__ __forceinline__ float4 normal4(uint4 w) {
    const float2 a = box_muller(w.x, w.y);
    const float2 b = box_muller(w.z, w.w);
    return make_float4(a.x, a.y, b.x, b.y);
}

__device__ __forceinline__ float4 noise4(uint32_t block, uint32_t node, uint32_t step, uint32_t tag,
                                         const PhiloxKeys& keys) {
    return normal4(philox4x32_10(make_uint4(block, node, step, tag), keys));
}

}  // namespace bgrpo
