// Counter-based Gaussian noise on the device: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11)
// and a float32 Box-Muller transform.  The stream definition (key, counter words, tags, uniform
// map, pairing) is the one stated at the top of bgrpo.h.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace bgrpo {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// Ten rounds; one round sends (c0,c1,c2,c3) to (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0))
// and the key advances by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c.x;
        const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * c.z;
        const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
        const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += kPhiloxW0;
        k1 += kPhiloxW1;
    }
    return c;
}

// u = ((x >> 9) + 0.5) * 2^-23, built without an integer-to-float conversion: the 23 kept bits become the
// mantissa of a float in [1, 2), and subtracting 1 - 2^-24 is exact.
__device__ __forceinline__ float uniform_open(uint32_t x) {
    return __uint_as_float((x >> 9) | 0x3f800000u) - 0.99999994f;
}

__device__ __forceinline__ float fast_sqrt(float x) {
    float y;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One Box-Muller pair from two words: (r cos 2 pi u_b, r sin 2 pi u_b), r = sqrt(-2 ln u_a).
//
// Accuracy (the result must stay within ~1e-4 of the exact value so that g * xi, g ~ 0.1, moves a
// latent by well under 1e-5):
//  * -2 ln u_a comes from the hardware log2 (absolute error 2^-22 for arguments in (0.5, 2), relative
//    2^-22 elsewhere).  An absolute error in r^2 becomes a large relative error in r only when r is tiny,
//    i.e. u_a within 2^-9 of 1; there w = 1 - u_a is exact in float32 and the series
//    -ln(1 - w) = w + w^2/2 + w^3/3 (truncation below 2e-9 relative) replaces the log.
//  * the angle is folded to (-pi, pi), where the hardware sine/cosine are good to about 4e-7 absolute,
//    and the sign change is absorbed into r.
__device__ __forceinline__ float2 box_muller(uint32_t wa, uint32_t wb) {
    const float ua = uniform_open(wa);
    const float ub = uniform_open(wb);
    const float w = 1.0f - ua;
    const float series = 2.0f * w * fmaf(w, fmaf(w, 0.33333334f, 0.5f), 1.0f);
    const float viaLog = -1.3862944f * __log2f(ua);          // -2 ln 2 * log2(u)
    const float r2 = (w < 0.001953125f) ? series : viaLog;
    const float nr = -fast_sqrt(r2);
    const float th = fmaf(ub, 6.2831855f, -3.1415927f);       // 2 pi u_b - pi
    float sn, cs;
    __sincosf(th, &sn, &cs);
    return make_float2(nr * cs, nr * sn);
}

__device__ __forceinline__ float4 normal4(uint4 w) {
    const float2 a = box_muller(w.x, w.y);
    const float2 b = box_muller(w.z, w.w);
    return make_float4(a.x, a.y, b.x, b.y);
}

__device__ __forceinline__ float4 noise4(uint32_t block, uint32_t node, uint32_t step, uint32_t tag,
                                         uint32_t k0, uint32_t k1) {
    return normal4(philox4x32_10(make_uint4(block, node, step, tag), k0, k1));
}

}  // namespace bgrpo
