/*
 * Oracle (test infrastructure): the neuroevolution algorithm's ask and tell
 * (paper Section 4, "Devising New Algorithms": ask generates a population of
 * parameters, tell reports the evaluation results back for the state update).
 * The algorithm is PGPE with symmetric (antithetic) sampling, the one solver the
 * paper's release ships (Section 5), with centred-rank fitness shaping and an Adam
 * ascent step on the centre (Section 2, "Modern ML Optimizers").  Sigma is constant.
 */
#include "oracle.h"
#include <math.h>
#include <stdlib.h>

void oracle_eps_row(uint64_t seed, uint32_t generation, uint32_t pair, uint32_t D, float* eps)
{
    /* stream 0; one Philox call serves four consecutive dimensions */
    for (uint32_t quad = 0; 4u * quad < D; ++quad) {
        uint32_t r[4];
        float z[4];
        oracle_stream_words(seed, 0u, generation, pair, quad, r);
        oracle_normal4(r, z);
        for (uint32_t i = 0; i < 4u && 4u * quad + i < D; ++i)
            eps[4u * quad + i] = z[i];
    }
}

void oracle_ask(uint64_t seed, uint32_t generation, uint32_t P, uint32_t D,
                const float* center, float sigma, float* theta, float* eps)
{
    float* row = (float*)malloc(sizeof(float) * (size_t)D);
    for (uint32_t j = 0; j < P / 2u; ++j) {
        oracle_eps_row(seed, generation, j, D, row);
        float* plus  = theta + (size_t)(2u * j) * D;
        float* minus = theta + (size_t)(2u * j + 1u) * D;
        for (uint32_t d = 0; d < D; ++d) {
            plus[d]  = fmaf( sigma, row[d], center[d]);
            minus[d] = fmaf(-sigma, row[d], center[d]);
            if (eps) eps[(size_t)j * D + d] = row[d];
        }
    }
    free(row);
}

int oracle_centered_rank(const float* fitness, uint32_t P, int32_t* rank, float* u)
{
    for (uint32_t m = 0; m < P; ++m)
        if (fitness[m] != fitness[m]) return 1;
    for (uint32_t m = 0; m < P; ++m) {
        int32_t below = 0;
        for (uint32_t k = 0; k < P; ++k) {
            if (fitness[k] < fitness[m]) below++;
            else if (fitness[k] == fitness[m] && k < m) below++;
        }
        rank[m] = below;
        u[m] = (float)below / (float)(P - 1u) - 0.5f;
    }
    return 0;
}

void oracle_gradient(const float* u, const float* eps, uint32_t P, uint32_t D,
                     double sigma, double* g)
{
    uint32_t H = P / 2u;
    for (uint32_t d = 0; d < D; ++d) {
        double acc = 0.0;
        for (uint32_t j = 0; j < H; ++j) {
            double w = (double)u[2u * j] - (double)u[2u * j + 1u];
            acc += w * (double)eps[(size_t)j * D + d];
        }
        g[d] = sigma / (double)P * acc;
    }
}

void oracle_adam(double* center, double* m, double* v, const double* g, uint32_t D,
                 uint32_t t, double lr, double beta1, double beta2, double adam_eps)
{
    double c1 = 1.0 - pow(beta1, (double)t);
    double c2 = 1.0 - pow(beta2, (double)t);
    for (uint32_t d = 0; d < D; ++d) {
        m[d] = beta1 * m[d] + (1.0 - beta1) * g[d];
        v[d] = beta2 * v[d] + (1.0 - beta2) * g[d] * g[d];
        double mhat = m[d] / c1;
        double vhat = v[d] / c2;
        center[d] += lr * mhat / (sqrt(vhat) + adam_eps);   /* ascent: fitness is maximised */
    }
}

/* ---- per-dimension sigma (PGPE keeps one standard deviation per parameter) ------------------ */

void oracle_ask_sigma(uint64_t seed, uint32_t generation, uint32_t P, uint32_t D,
                      const float* center, const float* sigma, float* theta, float* eps)
{
    float* row = (float*)malloc(sizeof(float) * (size_t)D);
    for (uint32_t j = 0; j < P / 2u; ++j) {
        oracle_eps_row(seed, generation, j, D, row);
        float* plus  = theta + (size_t)(2u * j) * D;
        float* minus = theta + (size_t)(2u * j + 1u) * D;
        for (uint32_t d = 0; d < D; ++d) {
            plus[d]  = fmaf( sigma[d], row[d], center[d]);
            minus[d] = fmaf(-sigma[d], row[d], center[d]);
            if (eps) eps[(size_t)j * D + d] = row[d];
        }
    }
    free(row);
}

void oracle_gradient_sigma(const float* u, const float* eps, uint32_t P, uint32_t D,
                           const double* sigma, double* g)
{
    uint32_t H = P / 2u;
    for (uint32_t d = 0; d < D; ++d) {
        double acc = 0.0;
        for (uint32_t j = 0; j < H; ++j)
            acc += ((double)u[2u * j] - (double)u[2u * j + 1u]) * (double)eps[(size_t)j * D + d];
        g[d] = sigma[d] / (double)P * acc;
    }
}

void oracle_sigma_gradient(const float* u, const float* eps, uint32_t P, uint32_t D,
                           const double* sigma, double* gs)
{
    uint32_t H = P / 2u;
    double b = 0.0;
    for (uint32_t m = 0; m < P; ++m) b += (double)u[m];
    b /= (double)P;
    for (uint32_t d = 0; d < D; ++d) {
        double acc = 0.0;
        for (uint32_t j = 0; j < H; ++j) {
            double s = 0.5 * ((double)u[2u * j] + (double)u[2u * j + 1u]) - b;
            double e = sigma[d] * (double)eps[(size_t)j * D + d];          /* the perturbation itself */
            acc += s * (e * e - sigma[d] * sigma[d]) / sigma[d];
        }
        gs[d] = acc / (double)H;
    }
}

void oracle_sigma_update(double* sigma, const double* gs, uint32_t D, double lr_sigma, double max_change)
{
    for (uint32_t d = 0; d < D; ++d) {
        double lo = sigma[d] * (1.0 - max_change), hi = sigma[d] * (1.0 + max_change);
        double s = sigma[d] + lr_sigma * gs[d];
        if (s < lo) s = lo;
        if (s > hi) s = hi;
        sigma[d] = s;
    }
}

void oracle_clipup(double* center, double* velocity, const double* g, uint32_t D,
                   double lr, double momentum, double max_speed)
{
    double gn = 0.0;
    for (uint32_t d = 0; d < D; ++d) gn += g[d] * g[d];
    gn = sqrt(gn);
    double vn = 0.0;
    for (uint32_t d = 0; d < D; ++d) {
        double step = gn > 0.0 ? lr * g[d] / gn : 0.0;
        velocity[d] = momentum * velocity[d] + step;
        vn += velocity[d] * velocity[d];
    }
    vn = sqrt(vn);
    double scale = vn > max_speed ? max_speed / vn : 1.0;
    for (uint32_t d = 0; d < D; ++d) {
        velocity[d] *= scale;
        center[d] += velocity[d];
    }
}
