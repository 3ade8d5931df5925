/*
 * Oracle (test infrastructure): counter-based random numbers.
 *
 * Philox4x32-10 as published by Salmon, Moraes, Dror and Shaw (SC'11), then the
 * uniform and normal transforms this library defines.  The paper only says that the
 * solver "generates a population of parameters" (Section 4, ask) and that roll-out
 * seeds are generated centrally (Section 2); the generator and transforms are this
 * repository's reading, chosen so that a CPU and a GPU produce the same bits: every
 * floating-point step is one correctly rounded fp32 operation (+, *, /, sqrt, fma).
 * Compile with -ffp-contract=off so that the compiler fuses nothing on its own.
 */
#include "oracle.h"
#include <math.h>
#include <string.h>

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {            /* Weyl sequence on the key between rounds */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void oracle_stream_words(uint64_t seed, uint32_t stream, uint32_t generation,
                         uint32_t row, uint32_t item, uint32_t out[4])
{
    uint32_t ctr[4] = { item, row, generation, stream };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    oracle_philox4x32_10(ctr, key, out);
}

float oracle_u_open(uint32_t r)
{
    /* 24 random bits, shifted into (0, 1]; both the conversion and the product are exact */
    return (float)((r >> 8) + 1u) * 0x1p-24f;
}

float oracle_u_half(uint32_t r)
{
    return (float)(r >> 8) * 0x1p-24f;
}

static uint32_t f32_bits(float x) { uint32_t b; memcpy(&b, &x, 4); return b; }
static float bits_f32(uint32_t b) { float x; memcpy(&x, &b, 4); return x; }

/*
 * ln(u) for a positive normal fp32 u.  Split u = m * 2^e with m in [sqrt(1/2), sqrt(2)) and
 * f = m - 1 (exact); ln m = f - f^2/2 + f^3 P(f) with a degree-7 polynomial P fitted to
 * (ln(1+f) - f + f^2/2)/f^3 on that interval (coefficients are part of the definition, given as
 * fp32 bit patterns).  The form keeps full relative accuracy as u -> 1, and needs no division.
 */
static const uint32_t LN_POLY_BITS[8] = {
    0x3EAAAAA9u, 0xBE800064u, 0x3E4CD0A6u, 0xBE2A6AA7u, 0x3E116E25u, 0xBE04D5F2u, 0x3E022C8Du, 0xBDA5EB80u
};

float oracle_ln_f32(float u)
{
    uint32_t b = f32_bits(u);
    int e = (int)(b >> 23) - 126;                         /* u = m * 2^e, m in [0.5, 1) */
    float m = bits_f32((b & 0x007FFFFFu) | 0x3F000000u);
    if (m < 0.70710678f) { m = m * 2.0f; e -= 1; }
    float f = m - 1.0f;
    float z = f * f;
    float p = bits_f32(LN_POLY_BITS[7]);
    for (int i = 6; i >= 0; --i) p = fmaf(p, f, bits_f32(LN_POLY_BITS[i]));
    float t = f * z;
    float h = 0.5f * z;
    float r = fmaf(t, p, -h);
    float lnm = f + r;
    return fmaf((float)e, 0.69314718f, lnm);
}

/*
 * cos and sin of 2*pi*v for v in [0,1).  w = 4v counts quarter turns; k = nearest
 * integer (ties to even), t = w - k is exact with |t| <= 1/2, x = t*(pi/2) lies in
 * [-pi/4, pi/4] where the Taylor polynomials below (sin to x^9, cos to x^10) are accurate to
 * fp32 rounding.
 */
void oracle_cossin_2pi_f32(float v, float* c_out, float* s_out)
{
    float w = 4.0f * v;
    float kf = rintf(w);
    float t = w - kf;
    float x = t * 1.57079637f;
    float z = x * x;

    float sp = 1.0f / 362880.0f;               /*  1/9!  */
    sp = fmaf(sp, z, -1.0f / 5040.0f);         /* -1/7!  */
    sp = fmaf(sp, z, 1.0f / 120.0f);           /*  1/5!  */
    sp = fmaf(sp, z, -1.0f / 6.0f);            /* -1/3!  */
    sp = fmaf(sp, z, 1.0f);
    float sn = x * sp;

    float cp = -1.0f / 3628800.0f;             /* -1/10! */
    cp = fmaf(cp, z, 1.0f / 40320.0f);         /*  1/8!  */
    cp = fmaf(cp, z, -1.0f / 720.0f);          /* -1/6!  */
    cp = fmaf(cp, z, 1.0f / 24.0f);            /*  1/4!  */
    cp = fmaf(cp, z, -0.5f);
    float cs = fmaf(cp, z, 1.0f);

    int q = ((int)kf) & 3;                      /* angle = q*pi/2 + x */
    float c, s;
    switch (q) {
        case 0:  c =  cs; s =  sn; break;
        case 1:  c = -sn; s =  cs; break;
        case 2:  c = -cs; s = -sn; break;
        default: c =  sn; s = -cs; break;
    }
    *c_out = c; *s_out = s;
}

void oracle_normal4(const uint32_t r[4], float z[4])
{
    for (int h = 0; h < 2; ++h) {
        float u = oracle_u_open(r[2 * h]);
        float v = oracle_u_half(r[2 * h + 1]);
        float lnu = oracle_ln_f32(u);
        float radius = sqrtf(-2.0f * lnu);
        float c, s;
        oracle_cossin_2pi_f32(v, &c, &s);
        z[2 * h]     = radius * c;
        z[2 * h + 1] = radius * s;
    }
}
