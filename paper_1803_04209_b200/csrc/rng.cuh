// Counter-based noise: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) and the basic
// Box-Muller transform (Box & Muller, 1958), computed in registers.
//
// Addressing.  One Philox call serves elements 4q..4q+3 of one (sample, stream, decision):
//   counter = (q, sample index, stream, decision number), key = (seed low, seed high).
// Stream t (0..lag) is guide step t, 0x100 the transition, 0x200 the emission.
// Output words (r0, r1) make the normals of elements 4q and 4q+1, (r2, r3) those of 4q+2 and 4q+3:
//   u1 = ((r_a >> 8) + 1) / 2^24 in (0, 1],  u2 = (r_b >> 8) / 2^24 in [0, 1)   (both exact in fp32)
//   e_even = sqrt(-2 ln u1) cos(2 pi u2),  e_odd = sqrt(-2 ln u1) sin(2 pi u2).
#pragma once
#include <cstdint>

namespace cutoff {

constexpr uint32_t kStreamTransition = 0x100u;
constexpr uint32_t kStreamEmission = 0x200u;

struct Philox4 {
    uint32_t x, y, z, w;
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  uint32_t k0, uint32_t k1) {
    constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
    constexpr uint32_t kWeylA = 0x9E3779B9u, kWeylB = 0xBB67AE85u;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const unsigned long long prod_a = static_cast<unsigned long long>(kMulA) * c0;   // one wide multiply each
        const unsigned long long prod_b = static_cast<unsigned long long>(kMulB) * c2;
        c0 = static_cast<uint32_t>(prod_b >> 32) ^ c1 ^ k0;
        c1 = static_cast<uint32_t>(prod_b);
        c2 = static_cast<uint32_t>(prod_a >> 32) ^ c3 ^ k1;
        c3 = static_cast<uint32_t>(prod_a);
        k0 += kWeylA;
        k1 += kWeylB;
    }
    return Philox4{c0, c1, c2, c3};
}

__device__ __forceinline__ void box_muller(uint32_t r_a, uint32_t r_b, float& e_cos, float& e_sin) {
    const float u1 = static_cast<float>((r_a >> 8) + 1u) * 0x1p-24f;
    const float two_u2 = static_cast<float>(r_b >> 8) * 0x1p-23f;
    const float radius = sqrtf(-2.0f * logf(u1));
    float s, c;
    sincospif(two_u2, &s, &c);
    e_cos = radius * c;
    e_sin = radius * s;
}

// The same transform with the hardware approximations (lg2, sqrt, sin, cos): each is accurate to
// about 1e-6 absolute on the ranges used here, except that sqrt(-2 ln u1) loses relative accuracy
// for the rare u1 within ~1e-3 of 1 (radius below ~0.05, absolute error still below ~6e-4).
// Used only where the surrounding arithmetic is tf32.  The angle is taken in [-pi, pi) -- the same
// point on the circle as 2 pi u2 -- where the sine / cosine units are most accurate.
__device__ __forceinline__ void box_muller_fast(uint32_t r_a, uint32_t r_b, float& e_cos, float& e_sin) {
    const float u1 = static_cast<float>((r_a >> 8) + 1u) * 0x1p-24f;
    const float angle = static_cast<float>(static_cast<int32_t>(r_b) >> 8) * (6.283185307179586f * 0x1p-24f);
    const float r2 = fmaxf(-1.3862943611198906f * __log2f(u1), 0.0f);     // -2 ln u1
    float radius;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(radius) : "f"(r2));
    e_cos = radius * __cosf(angle);
    e_sin = radius * __sinf(angle);
}

__device__ __forceinline__ float exp_half_fast(float logvar) {            // exp(logvar / 2)
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(logvar * 0.7213475204444817f));
    return r;
}

// Four standard normals for elements 4q..4q+3.
__device__ __forceinline__ void normal4(uint32_t q, uint32_t sample, uint32_t stream, uint32_t step,
                                        uint32_t seed_lo, uint32_t seed_hi, float out[4]) {
    const Philox4 r = philox4x32_10(q, sample, stream, step, seed_lo, seed_hi);
    box_muller(r.x, r.y, out[0], out[1]);
    box_muller(r.z, r.w, out[2], out[3]);
}

__device__ __forceinline__ void normal4_fast(uint32_t q, uint32_t sample, uint32_t stream, uint32_t step,
                                             uint32_t seed_lo, uint32_t seed_hi, float out[4]) {
    const Philox4 r = philox4x32_10(q, sample, stream, step, seed_lo, seed_hi);
    box_muller_fast(r.x, r.y, out[0], out[1]);
    box_muller_fast(r.z, r.w, out[2], out[3]);
}

}  // namespace cutoff
