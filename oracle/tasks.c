/*
 * Oracle (test infrastructure): the vectorised tasks and the roll-out loop (paper
 * Section 4, "Experimenting with More Tasks": stateless reset(keys)/step(state,
 * action); Section 2: the simulation manager generates the roll-out seeds and runs
 * the loop; Section 4: at the start of a roll-out every member of the population
 * sees identical observations).  The paper prints no task equations: the cart-pole
 * below is the standard uniform-rod cart-pole, the tanh-linear task is a synthetic
 * stand-in for a larger control workload; both are readings fixed by this
 * repository's design notes.
 */
#include "oracle.h"
#include <math.h>
#include <stdlib.h>

/* ---- cart-pole swing-up -------------------------------------------------------- */

/* state s = (x, x_dot, theta, theta_dot); theta = 0 is upright */
static void cartpole_deriv(const oracle_cartpole_params* p, const double s[4], double force,
                           double ds[4])
{
    double total = p->cart_mass + p->pole_mass;
    double l = p->pole_half_length;
    double sn = sin(s[2]), cs = cos(s[2]);
    double tmp = (force + p->pole_mass * l * s[3] * s[3] * sn) / total;
    double theta_acc = (p->gravity * sn - cs * tmp) /
                       (l * (4.0 / 3.0 - p->pole_mass * cs * cs / total));
    double x_acc = tmp - p->pole_mass * l * theta_acc * cs / total;
    ds[0] = s[1];
    ds[1] = x_acc;
    ds[2] = s[3];
    ds[3] = theta_acc;
}

void oracle_cartpole_step(const oracle_cartpole_params* p, double s[4], double force)
{
    double h = p->dt;
    if (p->integrator == 1) {                         /* explicit Euler */
        double k[4];
        cartpole_deriv(p, s, force, k);
        for (int i = 0; i < 4; ++i) s[i] += h * k[i];
        return;
    }
    /* classical fourth-order Runge-Kutta, force held over the step */
    double k1[4], k2[4], k3[4], k4[4], y[4];
    cartpole_deriv(p, s, force, k1);
    for (int i = 0; i < 4; ++i) y[i] = s[i] + 0.5 * h * k1[i];
    cartpole_deriv(p, y, force, k2);
    for (int i = 0; i < 4; ++i) y[i] = s[i] + 0.5 * h * k2[i];
    cartpole_deriv(p, y, force, k3);
    for (int i = 0; i < 4; ++i) y[i] = s[i] + h * k3[i];
    cartpole_deriv(p, y, force, k4);
    for (int i = 0; i < 4; ++i) s[i] += h / 6.0 * (k1[i] + 2.0 * k2[i] + 2.0 * k3[i] + k4[i]);
}

double oracle_cartpole_energy(const oracle_cartpole_params* p, const double s[4])
{
    double total = p->cart_mass + p->pole_mass;
    double l = p->pole_half_length, mp = p->pole_mass;
    return 0.5 * total * s[1] * s[1] + mp * l * s[1] * s[3] * cos(s[2])
         + (2.0 / 3.0) * mp * l * l * s[3] * s[3] + mp * p->gravity * l * cos(s[2]);
}

double oracle_cartpole_momentum(const oracle_cartpole_params* p, const double s[4])
{
    return (p->cart_mass + p->pole_mass) * s[1] + p->pole_mass * p->pole_half_length * s[3] * cos(s[2]);
}

void oracle_cartpole_reset(uint64_t seed, uint32_t generation, uint32_t episode,
                           float init_range, float s0[4])
{
    /* stream 1, row = episode, item 0: four uniforms in [-a, a) */
    uint32_t r[4];
    oracle_stream_words(seed, 1u, generation, episode, 0u, r);
    float n[4];
    for (int i = 0; i < 4; ++i)
        n[i] = fmaf(2.0f * init_range, oracle_u_half(r[i]), -init_range);
    s0[0] = n[0];
    s0[1] = n[1];
    s0[2] = 3.14159274f + n[2];          /* pole hanging down */
    s0[3] = n[3];
}

static double* widen(const float* x, uint32_t n)
{
    double* y = (double*)malloc(sizeof(double) * (size_t)n);
    for (uint32_t i = 0; i < n; ++i) y[i] = (double)x[i];
    return y;
}

double oracle_rollout_cartpole(const float* theta_row, uint32_t n_layers, const uint32_t* sizes,
                               double action_scale, const oracle_cartpole_params* p,
                               float init_range, uint64_t seed, uint32_t generation,
                               uint32_t E, uint32_t T, double* trace)
{
    double* params = widen(theta_row, oracle_mlp_param_count(n_layers, sizes));
    double total = 0.0;
    for (uint32_t e = 0; e < E; ++e) {
        float s0[4];
        oracle_cartpole_reset(seed, generation, e, init_range, s0);
        double s[4] = { s0[0], s0[1], s0[2], s0[3] };
        double ret = 0.0;
        for (uint32_t t = 0; t < T; ++t) {
            double obs[5] = { s[0], s[1], cos(s[2]), sin(s[2]), s[3] };
            double force;
            oracle_mlp_forward(params, n_layers, sizes, obs, &force, action_scale);
            oracle_cartpole_step(p, s, force);
            ret += cos(s[2]) * exp(-s[0] * s[0]);        /* reward on the post-step state */
            if (trace)
                for (int i = 0; i < 4; ++i) trace[((size_t)e * T + t) * 4 + i] = s[i];
        }
        total += ret;
    }
    free(params);
    return total / (double)E;
}

/* ---- tanh-linear control task --------------------------------------------------- */

static void normals_into(uint64_t seed, uint32_t stream, uint32_t generation, uint32_t row,
                         uint32_t count, float* dst)
{
    for (uint32_t quad = 0; 4u * quad < count; ++quad) {
        uint32_t r[4];
        float z[4];
        oracle_stream_words(seed, stream, generation, row, quad, r);
        oracle_normal4(r, z);
        for (uint32_t i = 0; i < 4u && 4u * quad + i < count; ++i) dst[4u * quad + i] = z[i];
    }
}

void oracle_tanh_linear_constants(uint64_t seed, float* A, float* B)
{
    /* stream 4, generation 0; row 0 = A (row-major 28x28), row 1 = B (row-major 28x8) */
    normals_into(seed, 4u, 0u, 0u, ORACLE_TL_NX * ORACLE_TL_NX, A);
    normals_into(seed, 4u, 0u, 1u, ORACLE_TL_NX * ORACLE_TL_NA, B);
    for (int i = 0; i < ORACLE_TL_NX * ORACLE_TL_NX; ++i) A[i] = A[i] * 0.170084015f;  /* 0.9/sqrt(28) */
    for (int i = 0; i < ORACLE_TL_NX * ORACLE_TL_NA; ++i) B[i] = B[i] * 0.353553385f;  /* 1/sqrt(8)    */
}

void oracle_tanh_linear_reset(uint64_t seed, uint32_t generation, uint32_t episode, float* x0)
{
    normals_into(seed, 1u, generation, episode, ORACLE_TL_NX, x0);
}

double oracle_rollout_tanh_linear(const float* theta_row, uint32_t n_layers, const uint32_t* sizes,
                                  double action_scale, const float* A, const float* B,
                                  uint64_t seed, uint32_t generation,
                                  uint32_t E, uint32_t T, double* trace)
{
    enum { NX = ORACLE_TL_NX, NA = ORACLE_TL_NA };
    double* params = widen(theta_row, oracle_mlp_param_count(n_layers, sizes));
    double total = 0.0;
    for (uint32_t e = 0; e < E; ++e) {
        float x0[NX];
        oracle_tanh_linear_reset(seed, generation, e, x0);
        double x[NX], xn[NX], a[NA];
        for (int i = 0; i < NX; ++i) x[i] = (double)x0[i];
        double ret = 0.0;
        for (uint32_t t = 0; t < T; ++t) {
            oracle_mlp_forward(params, n_layers, sizes, x, a, action_scale);
            double xx = 0.0, aa = 0.0;
            for (int i = 0; i < NX; ++i) xx += x[i] * x[i];
            for (int i = 0; i < NA; ++i) aa += a[i] * a[i];
            ret += -xx - 0.01 * aa;                      /* reward on (x_t, a_t) */
            for (int i = 0; i < NX; ++i) {
                double acc = 0.0;
                for (int k = 0; k < NX; ++k) acc += (double)A[i * NX + k] * x[k];
                for (int k = 0; k < NA; ++k) acc += (double)B[i * NA + k] * a[k];
                xn[i] = tanh(acc);
            }
            for (int i = 0; i < NX; ++i) x[i] = xn[i];
            if (trace)
                for (int i = 0; i < NX; ++i) trace[((size_t)e * T + t) * NX + i] = x[i];
        }
        total += ret;
    }
    free(params);
    return total / (double)E;
}
