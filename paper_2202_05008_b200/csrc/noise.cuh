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

struct PhiloxKey { uint32_t k0, k1; };

// counter = (item, row, generation, stream)
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               PhiloxKey key)
{
    uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
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

// ln(u), u a positive normal float: u = m 2^e with m in [sqrt(1/2), sqrt(2)), ln m = 2 atanh(s).
__device__ __forceinline__ float ln_rn(float u)
{
    const uint32_t bits = __float_as_uint(u);
    int e = static_cast<int>(bits >> 23) - 126;
    float m = __uint_as_float((bits & 0x007FFFFFu) | 0x3F000000u);
    if (m < __uint_as_float(0x3F3504F3u)) { m = __fadd_rn(m, m); e -= 1; }
    const float s = __fdiv_rn(__fadd_rn(m, -1.0f), __fadd_rn(m, 1.0f));
    const float z = __fmul_rn(s, s);
    float p = __uint_as_float(0x3DBA2E8Cu);                    // 1/11
    p = __fmaf_rn(p, z, __uint_as_float(0x3DE38E39u));         // 1/9
    p = __fmaf_rn(p, z, __uint_as_float(0x3E124925u));         // 1/7
    p = __fmaf_rn(p, z, __uint_as_float(0x3E4CCCCDu));         // 1/5
    p = __fmaf_rn(p, z, __uint_as_float(0x3EAAAAABu));         // 1/3
    p = __fmaf_rn(p, z, 1.0f);
    const float twice = __fmul_rn(2.0f, __fmul_rn(s, p));
    return __fmaf_rn(__int2float_rn(e), __uint_as_float(0x3F317218u), twice);
}

// (cos, sin)(2 pi v), v in [0,1): quarter-turn reduction, Taylor polynomials on [-pi/4, pi/4].
__device__ __forceinline__ void cossin_2pi_rn(float v, float& c, float& s)
{
    const float w = __fmul_rn(4.0f, v);
    const float kf = rintf(w);                                  // nearest, ties to even
    const float t = __fadd_rn(w, -kf);
    const float x = __fmul_rn(t, __uint_as_float(0x3FC90FDBu)); // pi/2
    const float z = __fmul_rn(x, x);

    float sp = __uint_as_float(0xB2D7322Bu);                    // -1/11!
    sp = __fmaf_rn(sp, z, __uint_as_float(0x3638EF1Du));        //  1/9!
    sp = __fmaf_rn(sp, z, __uint_as_float(0xB9500D01u));        // -1/7!
    sp = __fmaf_rn(sp, z, __uint_as_float(0x3C088889u));        //  1/5!
    sp = __fmaf_rn(sp, z, __uint_as_float(0xBE2AAAABu));        // -1/3!
    sp = __fmaf_rn(sp, z, 1.0f);
    const float sn = __fmul_rn(x, sp);

    float cp = __uint_as_float(0x310F76C7u);                    //  1/12!
    cp = __fmaf_rn(cp, z, __uint_as_float(0xB493F27Eu));        // -1/10!
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

// Box-Muller: (r.x, r.y) -> (z.x, z.y), (r.z, r.w) -> (z.z, z.w)
__device__ __forceinline__ float4 normal4(uint4 r)
{
    float4 z;
    {
        const float radius = __fsqrt_rn(__fmul_rn(-2.0f, ln_rn(uniform_open(r.x))));
        float c, s;
        cossin_2pi_rn(uniform_half(r.y), c, s);
        z.x = __fmul_rn(radius, c);
        z.y = __fmul_rn(radius, s);
    }
    {
        const float radius = __fsqrt_rn(__fmul_rn(-2.0f, ln_rn(uniform_open(r.z))));
        float c, s;
        cossin_2pi_rn(uniform_half(r.w), c, s);
        z.z = __fmul_rn(radius, c);
        z.w = __fmul_rn(radius, s);
    }
    return z;
}

__device__ __forceinline__ float4 stream_normal4(PhiloxKey key, uint32_t stream, uint32_t generation,
                                                 uint32_t row, uint32_t item)
{
    return normal4(philox4x32_10(item, row, generation, stream, key));
}

}  // namespace evo
