// Task arithmetic shared by the rollout kernels (fp32): the cart-pole swing-up equations with a
// classical RK4 step, and the seeded reset that every population member shares (paper
// Section 4: identical initial observations; Section 2: centrally generated roll-out seeds).
#pragma once
#include "internal.h"
#include "noise.cuh"

namespace evo {

struct CartpoleConst {
    float total_mass, pole_mass_length, gravity, length, dt, inv_total;
    float pole_mass;
};

__device__ __forceinline__ CartpoleConst cartpole_const(const float* tp)
{
    CartpoleConst c;
    c.total_mass = tp[EVO_CP_CART_MASS] + tp[EVO_CP_POLE_MASS];
    c.inv_total = 1.0f / c.total_mass;
    c.pole_mass = tp[EVO_CP_POLE_MASS];
    c.length = tp[EVO_CP_POLE_HALF_LENGTH];
    c.pole_mass_length = tp[EVO_CP_POLE_MASS] * tp[EVO_CP_POLE_HALF_LENGTH];
    c.gravity = tp[EVO_CP_GRAVITY];
    c.dt = tp[EVO_CP_DT];
    return c;
}

struct CpState { float x, xd, th, thd; };

// time derivative of (x, x', theta, theta') for the uniform-rod cart-pole, theta = 0 upright
__device__ __forceinline__ CpState cartpole_deriv(const CartpoleConst& c, const CpState& s, float force)
{
    float sn, cs;
    sincosf(s.th, &sn, &cs);
    const float tmp = (force + c.pole_mass_length * s.thd * s.thd * sn) * c.inv_total;
    const float th_acc = (c.gravity * sn - cs * tmp) /
                         (c.length * (4.0f / 3.0f - c.pole_mass * cs * cs * c.inv_total));
    const float x_acc = tmp - c.pole_mass_length * th_acc * cs * c.inv_total;
    return CpState{ s.xd, x_acc, s.thd, th_acc };
}

__device__ __forceinline__ CpState cp_axpy(const CpState& s, float h, const CpState& k)
{
    return CpState{ fmaf(h, k.x, s.x), fmaf(h, k.xd, s.xd), fmaf(h, k.th, s.th), fmaf(h, k.thd, s.thd) };
}

// classical RK4, force held over the step
__device__ __forceinline__ CpState cartpole_step(const CartpoleConst& c, const CpState& s, float force)
{
    const float h = c.dt;
    const CpState k1 = cartpole_deriv(c, s, force);
    const CpState k2 = cartpole_deriv(c, cp_axpy(s, 0.5f * h, k1), force);
    const CpState k3 = cartpole_deriv(c, cp_axpy(s, 0.5f * h, k2), force);
    const CpState k4 = cartpole_deriv(c, cp_axpy(s, h, k3), force);
    const float w = h * (1.0f / 6.0f);
    CpState n;
    n.x   = s.x   + w * (k1.x   + 2.0f * k2.x   + 2.0f * k3.x   + k4.x);
    n.xd  = s.xd  + w * (k1.xd  + 2.0f * k2.xd  + 2.0f * k3.xd  + k4.xd);
    n.th  = s.th  + w * (k1.th  + 2.0f * k2.th  + 2.0f * k3.th  + k4.th);
    n.thd = s.thd + w * (k1.thd + 2.0f * k2.thd + 2.0f * k3.thd + k4.thd);
    return n;
}

// seeded start shared by all members: (0, 0, pi, 0) + Uniform(-a, a)^4, stream 1, row = episode
__device__ __forceinline__ CpState cartpole_reset(const PhiloxKey& key, uint32_t generation, uint32_t episode,
                                                  float a)
{
    const uint4 r = philox4x32_10(0u, episode, generation, 1u, key);
    const float two_a = __fmul_rn(2.0f, a);
    CpState s;
    s.x   = __fmaf_rn(two_a, uniform_half(r.x), -a);
    s.xd  = __fmaf_rn(two_a, uniform_half(r.y), -a);
    s.th  = __fadd_rn(__uint_as_float(0x40490FDBu), __fmaf_rn(two_a, uniform_half(r.z), -a));
    s.thd = __fmaf_rn(two_a, uniform_half(r.w), -a);
    return s;
}


// ---- latency-trimmed variants for the tiled kernel ---------------------------------------------
// The roll-out is a serial chain per episode, so the task step's dependent-instruction latency
// sets the step time.  sin/cos by quarter-turn reduction (two-term pi/2) and short Taylor
// polynomials evaluated side by side (abs. error < 1e-7 for |theta| < 1e3), divisions by
// reciprocal approximation (2 ulp).

__device__ __forceinline__ void sincos_fast(float th, float& sn, float& cs)
{
    const float kf = rintf(th * 0.636619772f);
    float r = fmaf(kf, -1.57079637f, th);
    r = fmaf(kf, 4.37113883e-8f, r);
    const float z = r * r;
    float sp = fmaf(z, 2.75573192e-6f, -1.98412698e-4f);
    float cp = fmaf(z, 2.48015873e-5f, -1.38888889e-3f);
    sp = fmaf(sp, z, 8.33333333e-3f);
    cp = fmaf(cp, z, 4.16666667e-2f);
    sp = fmaf(sp, z, -1.66666667e-1f);
    cp = fmaf(cp, z, -0.5f);
    const float s0 = fmaf(sp * z, r, r);
    const float c0 = fmaf(cp, z, 1.0f);
    const int q = __float2int_rn(kf) & 3;
    const float a = (q & 1) ? s0 : c0;
    const float b = (q & 1) ? c0 : s0;
    cs = (q == 1 || q == 2) ? -a : a;
    sn = (q >= 2) ? -b : b;
}

// derivative with sin/cos of s.th supplied by the caller
__device__ __forceinline__ CpState cartpole_deriv_fast_sc(const CartpoleConst& c, const CpState& s, float force,
                                                          float sn, float cs)
{
    const float tmp = fmaf(c.pole_mass_length * s.thd * s.thd, sn, force) * c.inv_total;
    const float den = c.length * fmaf(-c.pole_mass * c.inv_total * cs, cs, 4.0f / 3.0f);
    const float th_acc = __fdividef(fmaf(c.gravity, sn, -cs * tmp), den);
    const float x_acc = fmaf(-c.pole_mass_length * c.inv_total * th_acc, cs, tmp);
    return CpState{ s.xd, x_acc, s.thd, th_acc };
}

__device__ __forceinline__ CpState cartpole_deriv_fast(const CartpoleConst& c, const CpState& s, float force)
{
    float sn, cs;
    sincos_fast(s.th, sn, cs);
    return cartpole_deriv_fast_sc(c, s, force, sn, cs);
}

// RK4 step; (sn, cs) = sin/cos of s.th, which a caller that has just computed the observation of s
// already holds (the first stage then needs no sin/cos of its own; same arithmetic, same bits)
__device__ __forceinline__ CpState cartpole_step_fast_sc(const CartpoleConst& c, const CpState& s, float force,
                                                         float sn, float cs)
{
    const float h = c.dt;
    // sin/cos at the inner stages by rotating (sn, cs) through the stage's small angle increment d
    // (Taylor to d^7 / d^8: error < 3e-6 even at |d| = 1, i.e. a pole speed of 100 rad/s at dt = 0.01)
    auto stage = [&](const CpState& q, float d) {
        const float z = d * d;
        float sd = fmaf(z, -1.98412698e-4f, 8.33333333e-3f);
        sd = fmaf(sd, z, -1.66666667e-1f);
        sd = fmaf(sd * z, d, d);
        float cd = fmaf(z, 2.48015873e-5f, -1.38888889e-3f);
        cd = fmaf(cd, z, 4.16666667e-2f);
        cd = fmaf(cd, z, -0.5f);
        cd = fmaf(cd, z, 1.0f);
        const float s2 = fmaf(sn, cd, cs * sd);
        const float c2 = fmaf(cs, cd, -sn * sd);
        return cartpole_deriv_fast_sc(c, q, force, s2, c2);
    };
    const CpState k1 = cartpole_deriv_fast_sc(c, s, force, sn, cs);
    const CpState k2 = stage(cp_axpy(s, 0.5f * h, k1), 0.5f * h * k1.th);
    const CpState k3 = stage(cp_axpy(s, 0.5f * h, k2), 0.5f * h * k2.th);
    const CpState k4 = stage(cp_axpy(s, h, k3), h * k3.th);
    const float w = h * (1.0f / 6.0f);
    CpState n;
    n.x   = fmaf(w, (k1.x   + k4.x)   + 2.0f * (k2.x   + k3.x),   s.x);
    n.xd  = fmaf(w, (k1.xd  + k4.xd)  + 2.0f * (k2.xd  + k3.xd),  s.xd);
    n.th  = fmaf(w, (k1.th  + k4.th)  + 2.0f * (k2.th  + k3.th),  s.th);
    n.thd = fmaf(w, (k1.thd + k4.thd) + 2.0f * (k2.thd + k3.thd), s.thd);
    return n;
}

__device__ __forceinline__ CpState cartpole_step_fast(const CartpoleConst& c, const CpState& s, float force)
{
    float sn, cs;
    sincos_fast(s.th, sn, cs);
    return cartpole_step_fast_sc(c, s, force, sn, cs);
}

}  // namespace evo
