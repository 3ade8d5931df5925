/*
 * CPU oracle for one evolution-strategy generation (ask -> rollout -> tell).
 *
 * TEST INFRASTRUCTURE ONLY.  This is the plain, slow, single-threaded restatement of
 * what the generation computes, used by the tests, by the smoke check and by the
 * benchmark's CPU-baseline leg.  The product (the CUDA library) never links, loads
 * or calls anything in this directory, and this directory shares no source, header,
 * table or helper with the CUDA sources.
 *
 * Arithmetic is fp64 except where a value is *defined* as an fp32 (or bf16) number:
 * the random normals, the sampled parameter matrix theta, the task's seeded initial
 * state and constants, the centred-rank weights, and the bf16 operand rounding of
 * the convolutional policy.  Those are computed in the defined precision with
 * single correctly-rounded IEEE operations and then widened.
 *
 * The paper (EvoJAX, GECCO'22) defines the structure -- a solver with ask/tell
 * (Section 4, "Devising New Algorithms"), a policy whose get_actions maps vectorised
 * task states and population parameters to actions (Section 4, "Exploring Novel
 * Policy Architectures"), a stateless vectorised task with reset/step (Section 4,
 * "Experimenting with More Tasks") and a roll-out loop run by the simulation manager
 * (Section 2) -- but prints no formulas.  The formulas here are the textbook ones
 * of the methods the paper names (PGPE with symmetric sampling, Adam) and the
 * readings fixed in this repository's design notes.
 *
 * Parity pins (tests marked "not gpu"): Philox known-answer vectors; Box-Muller
 * against libm in fp64 and against moments; antithetic-pair identity; rank is a
 * permutation and equals a sort; gradient against brute force from theta alone;
 * Adam against torch.optim.Adam; MLP against a numpy matmul; cart-pole energy and
 * momentum conservation, equilibria and small-angle period; tanh-linear recurrence
 * by hand; CNN against torch conv2d/max_pool2d/cross_entropy and the ln(10) case; the LSTM
 * seq2seq policy against torch.nn.LSTM + Linear + cross_entropy and the ln(12) case; its
 * queries against integer addition; the triangle painter against hand-counted coverage, closed-form
 * blending, vertex-order invariance and a barycentric rasteriser.
 * Parity unpinned (conventions only, nothing external fixes them): counter/stream
 * layout of the random numbers, the sign order inside an antithetic pair, the
 * observation order, reward timing, flatten order of the CNN, token codes and teacher forcing
 * of the seq2seq task.
 */
#ifndef ES_ORACLE_H
#define ES_ORACLE_H

#include <stdint.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- random numbers ------------------------------------------------------------ */

/* Philox4x32 with 10 rounds (Salmon et al., SC'11). */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* Counter convention of this library: key = seed (lo, hi);
 * counter = (item, row, generation, stream). */
void oracle_stream_words(uint64_t seed, uint32_t stream, uint32_t generation,
                         uint32_t row, uint32_t item, uint32_t out[4]);

float oracle_u_open(uint32_t r);   /* ((r>>8)+1) * 2^-24  in (0,1] */
float oracle_u_half(uint32_t r);   /* (r>>8) * 2^-24      in [0,1) */

/* fp32 natural log of u = k*2^-24 and fp32 (cos, sin) of 2*pi*v, each built from
 * single correctly rounded fp32 operations only. */
float oracle_ln_f32(float u);
void  oracle_cossin_2pi_f32(float v, float* c, float* s);

/* Box-Muller on four words: (r0,r1)->(z0,z1), (r2,r3)->(z2,z3). */
void oracle_normal4(const uint32_t r[4], float z[4]);

/* ---- solver: ask ---------------------------------------------------------------- */

/* eps[j][d] for one antithetic pair j: D standard normals of stream 0. */
void oracle_eps_row(uint64_t seed, uint32_t generation, uint32_t pair, uint32_t D, float* eps);

/* theta[2j] = fma(+sigma, eps_j, center), theta[2j+1] = fma(-sigma, eps_j, center), fp32.
 * theta is [P][D] dense; eps (may be NULL) is [P/2][D]. */
void oracle_ask(uint64_t seed, uint32_t generation, uint32_t P, uint32_t D,
                const float* center, float sigma, float* theta, float* eps);

/* ---- solver: tell --------------------------------------------------------------- */

/* rank[m] = #{k: f[k] < f[m] or (f[k] == f[m] and k < m)};
 * u[m] = (float)rank/(float)(P-1) - 0.5f.  Returns 1 if any fitness is NaN (outputs
 * then undefined), else 0. */
int oracle_centered_rank(const float* fitness, uint32_t P, int32_t* rank, float* u);

/* g[d] = (sigma/P) * sum_j (u[2j]-u[2j+1]) * eps[j][d], fp64. */
void oracle_gradient(const float* u, const float* eps, uint32_t P, uint32_t D,
                     double sigma, double* g);

/* One bias-corrected Adam ascent step (epsilon outside the root); t is the step
 * number after the increment (first call t = 1). */
void oracle_adam(double* center, double* m, double* v, const double* g, uint32_t D,
                 uint32_t t, double lr, double beta1, double beta2, double adam_eps);

/* ---- solver: per-dimension sigma and its PGPE update; ClipUp -------------------------- */

/* ask with a sigma vector: theta[2j][d] = fma(+sigma[d], eps, center[d]), and the mirrored member. */
void oracle_ask_sigma(uint64_t seed, uint32_t generation, uint32_t P, uint32_t D,
                      const float* center, const float* sigma, float* theta, float* eps);

/* g[d] = (sigma[d]/P) * sum_j (u[2j]-u[2j+1]) * eps[j][d]   (eps are the standard normals) */
void oracle_gradient_sigma(const float* u, const float* eps, uint32_t P, uint32_t D,
                           const double* sigma, double* g);

/* PGPE sigma gradient with symmetric sampling and baseline b = mean(u):
 * gs[d] = (1/H) * sum_j ((u[2j]+u[2j+1])/2 - b) * ((sigma[d] eps[j][d])^2 - sigma[d]^2) / sigma[d] */
void oracle_sigma_gradient(const float* u, const float* eps, uint32_t P, uint32_t D,
                           const double* sigma, double* gs);

/* sigma[d] += lr_sigma * gs[d], then clipped to [sigma_old (1 - max_change), sigma_old (1 + max_change)] */
void oracle_sigma_update(double* sigma, const double* gs, uint32_t D, double lr_sigma, double max_change);

/* ClipUp (Toklu et al. 2020), ascent: v = momentum v + lr g/|g|; if |v| > max_speed, v is scaled
 * back to that length; center += v. */
void oracle_clipup(double* center, double* velocity, const double* g, uint32_t D,
                   double lr, double momentum, double max_speed);

/* ---- policies ------------------------------------------------------------------- */

/* MLP: sizes[0..n_layers] (n_layers weight matrices). Flat parameters per layer:
 * W[out][in] row-major then b[out].  tanh after every layer, output times scale. */
void oracle_mlp_forward(const double* params, uint32_t n_layers, const uint32_t* sizes,
                        const double* x, double* y, double action_scale);
uint32_t oracle_mlp_param_count(uint32_t n_layers, const uint32_t* sizes);

/* CNN 28x28: conv(1->8,5x5,valid)+ReLU+pool2, conv(8->16,5x5,valid)+ReLU+pool2,
 * linear 256->10.  Returns -mean cross-entropy over the batch.  bf16_operands != 0
 * rounds the operands of the three contractions to bf16 (round to nearest even). */
double oracle_cnn_fitness(const float* params /*5994*/, const float* images /*[B][28][28]*/,
                          const int32_t* labels, uint32_t B, int bf16_operands);
void oracle_cnn_logits(const float* params, const float* image /*[28][28]*/,
                       int bf16_operands, double logits[10]);
float oracle_bf16_round(float x);

/* LSTM encoder-decoder on the addition task (paper Section 3, "Seq2Seq Learning"); conventions in
 * seq2seq.c.  Tokens: [B][2 nd + 1] encoder, [B][nd + 1] decoder inputs and targets.  Returns
 * minus the mean cross-entropy over all answer positions; *accuracy (may be NULL) receives the
 * fraction of positions whose arg-max token is right; logits_out (may be NULL) is [B][nd+1][12]. */
uint32_t oracle_seq2seq_param_count(uint32_t h);
void oracle_seq2seq_queries(uint64_t seed, uint32_t generation, uint32_t B, uint32_t nd,
                            int32_t* enc_tokens, int32_t* dec_tokens, int32_t* targets);
double oracle_seq2seq_fitness(const float* params, uint32_t h, uint32_t nd, uint32_t B,
                              const int32_t* enc_tokens, const int32_t* dec_tokens,
                              const int32_t* targets, int bf16_operands, double* accuracy,
                              double* logits_out);

/* Triangle painting (paper Section 3, "Concrete and Abstract Painting"); conventions in paint.c.
 * params: n_triangles x (x0 y0 x1 y1 x2 y2 r g b a); canvas and target are [H][W][3]. */
int  oracle_paint_inside(const float tri[6], float px, float py);
void oracle_paint_render(const float* params, uint32_t n_triangles, uint32_t W, uint32_t H,
                         double background, double* canvas);
double oracle_paint_fitness(const float* params, uint32_t n_triangles, uint32_t W, uint32_t H,
                            double background, const float* target, double* canvas /* scratch, output */);

/* ---- tasks ---------------------------------------------------------------------- */

typedef struct {
    double cart_mass, pole_mass, pole_half_length, gravity, dt;
    int    integrator;            /* 0 = classical RK4, 1 = explicit Euler */
} oracle_cartpole_params;

/* Seeded start: (0,0,pi,0) + Uniform(-a,a)^4, fp32, identical for all members. */
void   oracle_cartpole_reset(uint64_t seed, uint32_t generation, uint32_t episode,
                             float init_range, float s0[4]);
void   oracle_cartpole_step(const oracle_cartpole_params* p, double s[4], double force);
double oracle_cartpole_energy(const oracle_cartpole_params* p, const double s[4]);
double oracle_cartpole_momentum(const oracle_cartpole_params* p, const double s[4]);

/* Roll one member through E episodes of T steps; returns mean episode return.
 * trace (may be NULL) receives the post-step state, [E][T][4]. */
double oracle_rollout_cartpole(const float* theta_row, uint32_t n_layers, const uint32_t* sizes,
                               double action_scale, const oracle_cartpole_params* p,
                               float init_range, uint64_t seed, uint32_t generation,
                               uint32_t E, uint32_t T, double* trace);

/* Tanh-linear task: x' = tanh(A x + B a), reward -|x|^2 - 0.01 |a|^2 on (x_t, a_t). */
#define ORACLE_TL_NX 28
#define ORACLE_TL_NA 8
void   oracle_tanh_linear_constants(uint64_t seed, float* A /*[28][28]*/, float* B /*[28][8]*/);
void   oracle_tanh_linear_reset(uint64_t seed, uint32_t generation, uint32_t episode, float* x0);
double oracle_rollout_tanh_linear(const float* theta_row, uint32_t n_layers, const uint32_t* sizes,
                                  double action_scale, const float* A, const float* B,
                                  uint64_t seed, uint32_t generation,
                                  uint32_t E, uint32_t T, double* trace /*[E][T][28] or NULL*/);

#ifdef __cplusplus
}
#endif
#endif
