// Counter-based random numbers on the device: Philox4x32-10 (Salmon et al., SC'11), 24-bit
// uniforms and a Box-Muller transform whose every floating-point step is a single IEEE
// round-to-nearest fp32 operation (explicit *_rn intrinsics: the compiler may neither fuse
// nor approximate them), so that the same counters give the same bits on any conforming
// machine.  Used by ask (ES noise), by the regenerated-noise gradient and by task resets
// (the centrally generated roll-out seeds of the paper's Section 2).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace evo {

// The key with its schedule: round r uses (k0 + r W0, k1 + r W1), W = the Weyl increments.  The ten
// pairs are computed once where the key is made (on the host for the solver kernels, whose key is a
// launch parameter: the round keys then come straight out of the constant bank and the generator
// spends no instruction on the schedule).
struct PhiloxKey { uint32_t r[20]; };

__host__ __device__ __forceinline__ PhiloxKey philox_key(uint32_t k0, uint32_t k1)
{
    PhiloxKey k;
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        k.r[2 * i] = k0 + static_cast<uint32_t>(i) * 0x9E3779B9u;
        k.r[2 * i + 1] = k1 + static_cast<uint32_t>(i) * 0xBB67AE85u;
    }
    return k;
}

// counter = (item, row, generation, stream)
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKey& key)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;      // one wide multiply each
        const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
        const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
        const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
        c0 = hi1 ^ c1 ^ key.r[2 * r];
        c1 = lo1;
        c2 = hi0 ^ c3 ^ key.r[2 * r + 1];
        c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ float uniform_open(uint32_t r)   // (0, 1]
{
    return __fmul_rn(__uint2float_rn((r >> 8) + 1u), 5.9604644775390625e-08f);
}
__device__ __forceinline__ float uniform_half(uint32_t r)   // [0, 1)
{
    return __fmul_rn(__uint2float_rn(r >> 8), 5.9604644775390625e-08f);
}

// ln(k * 2^-24) for an integer k in [1, 2^24]: k = m 2^e with m in [sqrt(1/2), sqrt(2)), f = m - 1,
// ln m = f - f^2/2 + f^3 P(f), P of degree 7 (its coefficients are part of the definition of the
// generator).  Relative accuracy holds up to k = 2^24 (u = 1), and there is no division.
__device__ __forceinline__ float ln_of_u24(uint32_t k)
{
    const uint32_t bits = __float_as_uint(__uint2float_rn(k));            // exact: k <= 2^24
    int e = static_cast<int>(bits >> 23) - (126 + 24);                     // exponent of u = k 2^-24
    float m = __uint_as_float((bits & 0x007FFFFFu) | 0x3F000000u);         // [0.5, 1)
    if (m < __uint_as_float(0x3F3504F3u)) { m = __fadd_rn(m, m); e -= 1; }
    const float f = __fadd_rn(m, -1.0f);
    const float z = __fmul_rn(f, f);
    float p = __uint_as_float(0xBDA5EB80u);
    p = __fmaf_rn(p, f, __uint_as_float(0x3E022C8Du));
    p = __fmaf_rn(p, f, __uint_as_float(0xBE04D5F2u));
    p = __fmaf_rn(p, f, __uint_as_float(0x3E116E25u));
    p = __fmaf_rn(p, f, __uint_as_float(0xBE2A6AA7u));
    p = __fmaf_rn(p, f, __uint_as_float(0x3E4CD0A6u));
    p = __fmaf_rn(p, f, __uint_as_float(0xBE800064u));
    p = __fmaf_rn(p, f, __uint_as_float(0x3EAAAAA9u));
    const float t = __fmul_rn(f, z);
    const float h = __fmul_rn(0.5f, z);
    const float r = __fmaf_rn(t, p, -h);
    const float lnm = __fadd_rn(f, r);
    return __fmaf_rn(__int2float_rn(e), __uint_as_float(0x3F317218u), lnm);
}

// (cos, sin)(2 pi v) for v = j * 2^-24, j in [0, 2^24): quarter-turn reduction, Taylor polynomials
// (sin to x^9, cos to x^10) on [-pi/4, pi/4].
__device__ __forceinline__ void cossin_of_v24(uint32_t j, float& c, float& s)
{
    const float w = __fmul_rn(__uint2float_rn(j), 2.384185791015625e-07f);   // 4 v = j 2^-22, exact
    const float kf = rintf(w);                                  // nearest, ties to even
    const float t = __fadd_rn(w, -kf);
    const float x = __fmul_rn(t, __uint_as_float(0x3FC90FDBu)); // pi/2
    const float z = __fmul_rn(x, x);

    float sp = __uint_as_float(0x3638EF1Du);                    //  1/9!
    sp = __fmaf_rn(sp, z, __uint_as_float(0xB9500D01u));        // -1/7!
    sp = __fmaf_rn(sp, z, __uint_as_float(0x3C088889u));        //  1/5!
    sp = __fmaf_rn(sp, z, __uint_as_float(0xBE2AAAABu));        // -1/3!
    sp = __fmaf_rn(sp, z, 1.0f);
    const float sn = __fmul_rn(x, sp);

    float cp = __uint_as_float(0xB493F27Eu);                    // -1/10!
    cp = __fmaf_rn(cp, z, __uint_as_float(0x37D00D01u));        //  1/8!
    cp = __fmaf_rn(cp, z, __uint_as_float(0xBAB60B61u));        // -1/6!
    cp = __fmaf_rn(cp, z, __uint_as_float(0x3D2AAAABu));        //  1/4!
    cp = __fmaf_rn(cp, z, -0.5f);
    const float cs = __fmaf_rn(cp, z, 1.0f);

    const int q = __float2int_rn(kf) & 3;
    const float a = (q & 1) ? sn : cs;                          // |cos| source
    const float b = (q & 1) ? cs : sn;                          // |sin| source
    c = (q == 1 || q == 2) ? -a : a;
    s = (q >= 2) ? -b : b;
}

// Box-Muller: (r.x, r.y) -> (z.x, z.y), (r.z, r.w) -> (z.z, z.w);
// radius = sqrt(-2 ln u), u = ((r_even >> 8) + 1) 2^-24; angle = 2 pi (r_odd >> 8) 2^-24
__device__ __forceinline__ float4 normal4(uint4 r)
{
    float4 z;
    {
        const float radius = __fsqrt_rn(__fmul_rn(-2.0f, ln_of_u24((r.x >> 8) + 1u)));
        float c, s;
        cossin_of_v24(r.y >> 8, c, s);
        z.x = __fmul_rn(radius, c);
        z.y = __fmul_rn(radius, s);
    }
    {
        const float radius = __fsqrt_rn(__fmul_rn(-2.0f, ln_of_u24((r.z >> 8) + 1u)));
        float c, s;
        cossin_of_v24(r.w >> 8, c, s);
        z.z = __fmul_rn(radius, c);
        z.w = __fmul_rn(radius, s);
    }
    return z;
}

__device__ __forceinline__ float4 stream_normal4(const PhiloxKey& key, uint32_t stream, uint32_t generation,
                                                 uint32_t row, uint32_t item)
{
    return normal4(philox4x32_10(item, row, generation, stream, key));
}

}  // namespace evo
