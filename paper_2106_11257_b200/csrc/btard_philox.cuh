// Device-side GetRandomVector (Alg. 6 line 5): Philox4x32-10 words mapped to standard normals.
//
// z is never stored on the verification path; each group of four coordinates is produced in
// registers from the counter (q, partition, k, tag) and the 64-bit seed as key.  The word -> normal
// map is a Box-Muller written only with IEEE single-precision add, multiply, fused multiply-add
// and square root in a fixed order, so its results are a function of the words alone.
#pragma once
#include <cstdint>

namespace btard {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;   // Salmon et al., SC'11: multipliers
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;   // Weyl key increments
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;
constexpr uint32_t kCounterTag = 0x42544152u; // fourth counter word of every z block

struct uint4x { uint32_t x, y, z, w; };

__device__ __forceinline__ uint4x philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        // one 32 x 32 -> 64 bit product per multiplier; the round keys k + r W are loop-invariant
        // expressions of the seed, which the compiler hoists out of the caller's tile loop
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ (k0 + (uint32_t)r * kPhiloxW0);
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ (k1 + (uint32_t)r * kPhiloxW1);
        c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
    }
    return uint4x{c0, c1, c2, c3};
}

// Two words -> two N(0,1) values.
//   u = ((a >> 8) + 1) 2^-24,  t = -ln u  (ln by exponent split + polynomial),
//   y = ((b >> 6 & 0xFFFFFF) + 1/2) 2^-24 - 1/2,  S = sin(pi y / 2),  C = cos(pi y / 2),
//   (n0, n1) = sqrt(t) (C - S, C + S); bits 31 and 30 of b give the signs.
__device__ __forceinline__ void normal_pair(uint32_t a, uint32_t b, float& n0, float& n1)
{
    const uint32_t i = (a >> 8) + 1u;
    const uint32_t bits = __float_as_uint(__uint2float_rn(i));
    const uint32_t e = (bits - 0x3F3504F3u) >> 23;
    const float m = __uint_as_float(bits - (e << 23));
    const float x = __fadd_rn(m, -1.0f);
    float q = 0x1.eaf59cp-4f;
    q = __fmaf_rn(q, x, -0x1.803d52p-3f);
    q = __fmaf_rn(q, x, 0x1.a3b028p-3f);
    q = __fmaf_rn(q, x, -0x1.fde802p-3f);
    q = __fmaf_rn(q, x, 0x1.5526b4p-2f);
    q = __fmaf_rn(q, x, -0x1.0001f2p-1f);
    const float x2 = __fmul_rn(x, x);
    const float lnm = __fmaf_rn(x2, q, x);
    float t = __fmaf_rn(__int2float_rn(24 - (int)e), 0x1.62e43p-1f, -lnm);
    t = fmaxf(t, 0.0f);
    const float r = __fsqrt_rn(t);

    const uint32_t j = (b >> 6) & 0xFFFFFFu;
    const float y = __fmaf_rn(__uint2float_rn(j), 0x1p-24f, -0x1.fffffep-2f);
    const float z = __fmul_rn(y, y);
    float s = 0x1.3e202ap-4f;
    s = __fmaf_rn(s, z, -0x1.4a9ac4p-1f);
    s = __fmaf_rn(s, z, 0x1.921f32p+0f);
    s = __fmul_rn(s, y);
    float c = -0x1.4e5ed6p-6f;
    c = __fmaf_rn(c, z, 0x1.03af5cp-2f);
    c = __fmaf_rn(c, z, -0x1.3bd392p+0f);
    c = __fmaf_rn(c, z, 1.0f);
    const float a0 = __fmul_rn(r, __fadd_rn(c, -s));
    const float a1 = __fmul_rn(r, __fadd_rn(c, s));
    n0 = __uint_as_float(__float_as_uint(a0) ^ (b & 0x80000000u));
    n1 = __uint_as_float(__float_as_uint(a1) ^ ((b << 1) & 0x80000000u));
}

// Coordinates 4q .. 4q+3 of z_k of partition p.
__device__ __forceinline__ float4 z_quad(uint32_t q, uint32_t p, uint32_t k, uint32_t seed_lo,
                                         uint32_t seed_hi)
{
    const uint4x w = philox4x32_10(q, p, k, kCounterTag, seed_lo, seed_hi);
    float4 z;
    normal_pair(w.x, w.y, z.x, z.y);
    normal_pair(w.z, w.w, z.z, z.w);
    return z;
}

}  // namespace btard
