// Device-side GetRandomVector (Alg. 6): Philox4x32-10 words mapped to standard normals.
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

// Two words (a, b) -> two N(0,1) values:
//   u = ((a >> 8) + 1) 2^-24,  t = -ln u  (ln by exponent split + polynomial),
//   y = ((b >> 6 & 0xFFFFFF) + 1/2) 2^-24 - 1/2,  S = sin(pi y / 2),  C = cos(pi y / 2),
//   (n0, n1) = sqrt(t) (C - S, C + S); bits 31 and 30 of b give the signs.
// A Philox block holds two such word pairs, and both are mapped at once:
// sm_100 has packed single-precision instructions (add / mul / fma .f32x2: two IEEE operations, each
// rounded exactly like its scalar form), so the two word pairs of a Philox block share every
// floating-point step of the map; every lane sees the scalar operations in the scalar order.
__device__ __forceinline__ uint64_t pk2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t pk_add(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t pk_sub(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t pk_mul(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t pk_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t pk_const(float c) { return pk2(c, c); }

// Four words -> four N(0,1) values: (w.x, w.y) -> (z.x, z.y), (w.z, w.w) -> (z.z, z.w).
__device__ __forceinline__ float4 normal_quad(const uint4x w)
{
    const uint32_t i0 = (w.x >> 8) + 1u, i1 = (w.z >> 8) + 1u;
    const uint32_t b0 = __float_as_uint(__uint2float_rn(i0)), b1 = __float_as_uint(__uint2float_rn(i1));
    const uint32_t e0 = (b0 - 0x3F3504F3u) >> 23, e1 = (b1 - 0x3F3504F3u) >> 23;
    const uint64_t m = pk2(__uint_as_float(b0 - (e0 << 23)), __uint_as_float(b1 - (e1 << 23)));
    const uint64_t x = pk_add(m, pk_const(-1.0f));
    uint64_t q = pk_const(0x1.eaf59cp-4f);
    q = pk_fma(q, x, pk_const(-0x1.803d52p-3f));
    q = pk_fma(q, x, pk_const(0x1.a3b028p-3f));
    q = pk_fma(q, x, pk_const(-0x1.fde802p-3f));
    q = pk_fma(q, x, pk_const(0x1.5526b4p-2f));
    q = pk_fma(q, x, pk_const(-0x1.0001f2p-1f));
    // -ln m = fma(-(x x), q, -x): rounding to nearest is symmetric, so negating both inputs of the
    // scalar form's fma(x x, q, x) negates its result exactly
    const uint64_t nx = pk_sub(pk_const(1.0f), m);
    const uint64_t nx2 = pk_mul(nx, x);
    const uint64_t nlnm = pk_fma(nx2, q, nx);
    const uint64_t ef = pk2(__int2float_rn(24 - (int)e0), __int2float_rn(24 - (int)e1));
    const uint64_t t = pk_fma(ef, pk_const(0x1.62e43p-1f), nlnm);
    float t0, t1;
    upk2(t, t0, t1);
    const uint64_t r = pk2(__fsqrt_rn(fmaxf(t0, 0.0f)), __fsqrt_rn(fmaxf(t1, 0.0f)));

    const uint32_t j0 = (w.y >> 6) & 0xFFFFFFu, j1 = (w.w >> 6) & 0xFFFFFFu;
    const uint64_t y = pk_fma(pk2(__uint2float_rn(j0), __uint2float_rn(j1)), pk_const(0x1p-24f),
                              pk_const(-0x1.fffffep-2f));
    const uint64_t z = pk_mul(y, y);
    uint64_t s = pk_const(0x1.3e202ap-4f);
    s = pk_fma(s, z, pk_const(-0x1.4a9ac4p-1f));
    s = pk_fma(s, z, pk_const(0x1.921f32p+0f));
    {
        // This product feeds C - S and C + S.  As a packed multiply the assembler (CUDA 12.9) merges it
        // into those two and rounds once instead of twice; the scalar intrinsic is never merged.
        float s0, s1, y0, y1;
        upk2(s, s0, s1);
        upk2(y, y0, y1);
        s = pk2(__fmul_rn(s0, y0), __fmul_rn(s1, y1));
    }
    uint64_t c = pk_const(-0x1.4e5ed6p-6f);
    c = pk_fma(c, z, pk_const(0x1.03af5cp-2f));
    c = pk_fma(c, z, pk_const(-0x1.3bd392p+0f));
    c = pk_fma(c, z, pk_const(1.0f));
    float a00, a10, a01, a11;                          // a<which normal><which pair>
    upk2(pk_mul(r, pk_sub(c, s)), a00, a01);
    upk2(pk_mul(r, pk_add(c, s)), a10, a11);
    float4 out;
    out.x = __uint_as_float(__float_as_uint(a00) ^ (w.y & 0x80000000u));
    out.y = __uint_as_float(__float_as_uint(a10) ^ ((w.y << 1) & 0x80000000u));
    out.z = __uint_as_float(__float_as_uint(a01) ^ (w.w & 0x80000000u));
    out.w = __uint_as_float(__float_as_uint(a11) ^ ((w.w << 1) & 0x80000000u));
    return out;
}

// Coordinates 4q .. 4q+3 of z_k of partition p.
__device__ __forceinline__ float4 z_quad(uint32_t q, uint32_t p, uint32_t k, uint32_t seed_lo,
                                         uint32_t seed_hi)
{
    return normal_quad(philox4x32_10(q, p, k, kCounterTag, seed_lo, seed_hi));
}

}  // namespace btard
