/*
 * evo.h -- C-ABI of the B200 (sm_100a) library for one evolution-strategy generation:
 *
 *     evo_ask      sample the whole population   theta[2j], theta[2j+1] = center +- sigma*eps_j
 *     evo_rollout  evaluate every member         fitness[m] = mean episode return of policy(theta[m])
 *     evo_tell     update the search distribution  centred ranks -> ES gradient -> Adam ascent
 *
 * The split follows the component interfaces of the EvoJAX paper, Section 4 ("Extending
 * EvoJAX"): the algorithm's ask/tell ("Devising New Algorithms"), the policy's get_actions
 * over the whole population ("Exploring Novel Policy Architectures") and the stateless
 * vectorised task's reset/step ("Experimenting with More Tasks"); the roll-out loop and the
 * central generation of roll-out seeds are the simulation manager's job (Section 2).  The
 * paper prints no formulas; the ones quoted below are the textbook PGPE (symmetric sampling)
 * and Adam definitions the paper names (Sections 2 and 5).
 *
 * Conventions for every call
 *   - All pointers named d_* are DEVICE pointers owned by the caller; everything else is host
 *     memory.  The library never allocates or frees device memory, and launches all work on the
 *     CUDA stream given to evo_create (a cudaStream_t passed as void*).
 *   - No call synchronises the device except evo_sync_status.  Device-side conditions (a NaN
 *     fitness) are recorded in a status word inside the workspace and reported there.
 *   - Every call returns an evo_status; nothing prints, aborts or throws.
 *   - One solver = one stream = one host thread at a time.
 *   - Notation: P = pop_size (even), H = P/2 antithetic pairs, D = param_dim,
 *     ldD = D rounded up to a multiple of 32 floats (row pitch), E = episodes, T = horizon.
 */
#ifndef EVO_H
#define EVO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct evo_solver evo_solver;   /* opaque, host memory, freed by evo_destroy */

typedef enum {
    EVO_OK = 0,
    EVO_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, bad size, bad enum            */
    EVO_ERR_BAD_ORDER   = 2,   /* e.g. evo_tell before evo_ask                              */
    EVO_ERR_WORKSPACE   = 3,   /* workspace too small                                       */
    EVO_ERR_CUDA        = 4,   /* a CUDA runtime call or launch failed                      */
    EVO_ERR_NONFINITE   = 5,   /* a NaN fitness reached evo_tell; that update was skipped   */
    EVO_ERR_TIMEOUT     = 6,   /* a bounded device-side wait gave up                        */
    EVO_ERR_UNSUPPORTED = 7    /* valid request this build has no kernel for                */
} evo_status;

enum { EVO_NOISE_STORED = 0, EVO_NOISE_REGENERATED = 1 };
enum { EVO_POLICY_NONE = 0, EVO_POLICY_MLP = 1, EVO_POLICY_CNN_28 = 2, EVO_POLICY_LSTM_SEQ2SEQ = 3 };
enum { EVO_TASK_NONE = 0, EVO_TASK_CARTPOLE = 1, EVO_TASK_TANH_LINEAR = 2, EVO_TASK_SUPERVISED = 3,
       EVO_TASK_SEQ2SEQ_ADD = 4, EVO_TASK_PAINT = 5 };
/* Roll-out kernel of the control tasks.  GENERIC: runtime shapes, any MLP.  TILED: the fp32-pipe
 * kernels with the weights in registers (two hidden layers, each at most as wide as a compiled shape:
 * 16/32/64/128 for the cart-pole, 128 for the tanh-linear task); UNSUPPORTED at evo_rollout if none
 * fits.  AUTO: for the tanh-linear task with hidden widths <= 128 the tensor-core kernel (wide layers
 * as pairs of fp16 numbers on tcgen05, fp32-accurate; weights of those layers beyond +-65,504 are
 * clamped), else TILED where it fits, else GENERIC. */
enum { EVO_ROLLOUT_AUTO = 0, EVO_ROLLOUT_GENERIC = 1, EVO_ROLLOUT_TILED = 2 };
enum { EVO_OPT_ADAM = 0, EVO_OPT_CLIPUP = 1 };
enum { EVO_SIGMA_CONSTANT = 0, EVO_SIGMA_PGPE = 1 };
/* evo_config.debug_flags.  DROP_COMPLETION: the roll-out kernels leave out the asynchronous
 * completion their first bounded wait depends on (the copy of a member's parameter row; in the
 * tensor-core control kernel the commit of the first batch of MMAs; in the tensor-core CNN the
 * copy of a block's first group of activations), so that wait must run out: every block raises
 * EVO_ERR_TIMEOUT, reports NaN as its return and leaves by itself, with nothing left in flight.  It exists so that the time-out path can be tested without disturbing
 * the device. */
enum { EVO_DEBUG_DROP_COMPLETION = 1 };

/* indices into evo_config.task_param for EVO_TASK_CARTPOLE */
enum { EVO_CP_CART_MASS = 0, EVO_CP_POLE_MASS = 1, EVO_CP_POLE_HALF_LENGTH = 2, EVO_CP_GRAVITY = 3,
       EVO_CP_DT = 4, EVO_CP_INIT_RANGE = 5 };

/* index into evo_config.task_param for EVO_TASK_SEQ2SEQ_ADD: digits per operand, 1..4 */
enum { EVO_S2S_DIGITS = 0 };

/* indices into evo_config.task_param for EVO_TASK_PAINT: canvas width and height in pixels, grey
 * level of the empty canvas */
enum { EVO_PAINT_WIDTH = 0, EVO_PAINT_HEIGHT = 1, EVO_PAINT_BACKGROUND = 2 };

#define EVO_MAX_LAYERS 8

typedef struct evo_config {
    uint32_t struct_size;          /* sizeof(evo_config), checked                               */
    uint32_t pop_size;             /* P, even, >= 2                                             */
    uint64_t seed;                 /* Philox key of every random stream of this solver          */
    uint32_t param_dim;            /* D, 1 .. 2^30                                              */
    uint32_t noise_mode;           /* EVO_NOISE_*: keep eps[H][ldD] from ask, or recompute it   */
    float    sigma;                /* > 0, constant                                             */
    float    lr;                   /* Adam step size                                            */
    float    beta1, beta2, adam_eps;   /* 0 selects 0.9 / 0.999 / 1e-8                          */
    uint32_t policy_kind;          /* EVO_POLICY_*                                              */
    uint32_t n_layers;             /* MLP: number of weight matrices, 1..EVO_MAX_LAYERS         */
    uint32_t layer_sizes[EVO_MAX_LAYERS + 1];  /* MLP widths, input first; LSTM: [0] = hidden   */
    float    action_scale;         /* MLP output = scale * tanh(.)                              */
    uint32_t task_kind;            /* EVO_TASK_*; NONE = caller computes fitness itself         */
    uint32_t episodes;             /* E >= 1 (control tasks)                                    */
    uint32_t horizon;              /* T >= 1 (control tasks)                                    */
    uint32_t batch;                /* images (supervised) or queries (seq2seq) per member       */
    uint32_t trace_steps;          /* leading steps recorded when evo_rollout gets d_trace, <= T */
    uint32_t rollout_kernel;       /* EVO_ROLLOUT_*: AUTO picks the fastest kernel that fits    */
    float    task_param[16];       /* EVO_CP_* / EVO_S2S_* / EVO_PAINT_* by task; else unused   */
    uint32_t optimizer;            /* EVO_OPT_*: how the centre follows the ES gradient         */
    float    clipup_momentum;      /* ClipUp: 0 selects 0.9                                     */
    float    clipup_max_speed;     /* ClipUp: 0 selects 2 * lr                                  */
    uint32_t sigma_mode;           /* EVO_SIGMA_*: keep sigma, or adapt it per dimension (PGPE) */
    float    sigma_lr;             /* PGPE sigma step size, 0 selects 0.1                       */
    float    sigma_max_change;     /* largest relative change of sigma per tell, 0 selects 0.2  */
    uint32_t shard_first_pair;     /* multi-GPU: first antithetic pair this solver owns         */
    uint32_t shard_pairs;          /* multi-GPU: pairs it owns; 0 = the whole population        */
    uint32_t wait_cycles_log2;     /* a device-side wait gives up after 2^n SM clocks and raises
                                      EVO_ERR_TIMEOUT; 0 selects 31 (about a second), else 10..40 */
    uint32_t debug_flags;          /* EVO_DEBUG_* bits, 0 in production                          */
} evo_config;

/* Bytes of device workspace a solver with this configuration needs.  Pure host function. */
evo_status evo_workspace_bytes(const evo_config* cfg, size_t* bytes);

/*
 * Create a solver.  d_workspace: device memory, 256-byte aligned, at least
 * evo_workspace_bytes() long, owned by the caller and kept alive until evo_destroy.
 * cuda_stream: a cudaStream_t (NULL = default stream).  Enqueues the initialisation (centre,
 * Adam moments = 0, task constants) on the stream; generation and Adam step start at 0.
 * Errors: INVALID_ARG (bad config / pointer / alignment), WORKSPACE, UNSUPPORTED, CUDA.
 */
evo_status evo_create(const evo_config* cfg, void* d_workspace, size_t workspace_bytes,
                      void* cuda_stream, evo_solver** out);

/*
 * ask (paper Section 4, NEAlgorithm.ask; PGPE symmetric sampling, Section 5).  For pair j and
 * dimension d, eps[j][d] ~ N(0,1) from the counter-based generator at (seed, generation);
 * theta[2j][d] = fma(+sigma, eps, center[d]), theta[2j+1][d] = fma(-sigma, eps, center[d]).
 * Returns the device pointer of theta[P][ldD] (fp32, row-major, padding columns zero), which
 * lives in the workspace and is valid until the next evo_ask, and its row pitch in floats.
 */
evo_status evo_ask(evo_solver* s, const float** d_theta, size_t* ld_theta);

/*
 * rollout (paper Sections 2 and 4: the simulation manager's loop of PolicyNetwork.get_actions
 * and VectorizedTask.step over the population; supervised learning is a single-step task,
 * Section 3).  Evaluates all P members of d_theta (NULL = the matrix of the last evo_ask; a
 * caller matrix must be [P][ldD] with the same pitch, 16-byte aligned) and writes
 * d_fitness[P] (fp32).  Control tasks: E episodes of T steps per member from seeded initial
 * states shared by all members; fitness = mean episode return.  Supervised task: fitness =
 * -mean cross-entropy on the batch bound with evo_set_batch.  Seq2seq task: -mean cross-entropy of
 * the answer digits on `batch` queries the library draws itself.  Painting task (policy NONE: the
 * parameter row is param_dim / 10 triangles x0 y0 x1 y1 x2 y2 r g b a): -mean squared distance of
 * the painted canvas to the image bound with evo_set_target.
 * d_trace: NULL, or [P][E][trace_steps][state_dim] floats (16-byte aligned) receiving the
 * post-step task state of the first trace_steps steps (state_dim = 4 cart-pole: x, x', theta,
 * theta'; 28 tanh-linear); control tasks require trace_steps <= horizon at evo_create.
 * Errors: BAD_ORDER (d_theta NULL before any ask; supervised without a batch), INVALID_ARG,
 * UNSUPPORTED (task NONE), CUDA.
 */
evo_status evo_rollout(evo_solver* s, const float* d_theta, float* d_fitness, float* d_trace);

/*
 * tell (paper Section 4, NEAlgorithm.tell; Section 2 "Modern ML Optimizers").  With
 * rank_m = #{k: f_k < f_m or (f_k == f_m and k < m)} and u_m = rank_m/(P-1) - 1/2:
 *   g[d] = (sigma/P) * sum_j (u[2j] - u[2j+1]) * eps[j][d]
 *   t += 1;  m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g^2
 *   center += lr * (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + adam_eps)          (ascent)
 * eps is the noise of the matching evo_ask (read back in STORED mode, recomputed from the
 * counters in REGENERATED mode).  sigma is kept per dimension (all equal to cfg.sigma at
 * start): ask uses sigma[d], and the gradient above is scaled by sigma[d].
 * optimizer = EVO_OPT_CLIPUP replaces the Adam lines by ClipUp (the optimiser the paper's PGPE
 * reference pairs it with, Section 5): vel = momentum vel + lr g/|g|; if |vel| > max_speed it is
 * scaled back to that length; center += vel (vel lives in the first-moment buffer).
 * sigma_mode = EVO_SIGMA_PGPE also adapts sigma (PGPE with symmetric sampling, Section 5):
 *   gs[d] = (sigma[d]/H) * sum_j ((u[2j] + u[2j+1])/2) * (eps[j][d]^2 - 1)
 *   sigma[d] += sigma_lr * gs[d], limited to a relative change of +-sigma_max_change per tell.
 * Advances the generation.  A NaN in d_fitness[P] skips the update (centre, moments, sigma, t
 * unchanged) and raises EVO_ERR_NONFINITE at the next evo_sync_status.  Not available on a
 * sharded solver (shard_pairs > 0: EVO_ERR_UNSUPPORTED), which uses evo_tell_begin / _end.
 * Errors: BAD_ORDER (no ask since the last tell), INVALID_ARG, UNSUPPORTED, CUDA.
 */
evo_status evo_tell(evo_solver* s, const float* d_fitness);

/*
 * Sharded generation (paper Section 2, "Device Parallelism": the population is spread over the
 * accelerators).  A solver created with shard_pairs > 0 owns pairs [shard_first_pair,
 * shard_first_pair + shard_pairs) of a population of pop_size members: evo_ask returns only its
 * 2*shard_pairs members (their noise comes from the global pair index, so no noise is ever
 * exchanged), evo_rollout scores them into d_fitness[2*shard_pairs], and evo_tell is replaced by
 *   evo_tell_begin(s, d_fitness_all)  d_fitness_all[pop_size] in global member order (the caller
 *                                     all-gathers the shards' fitness): ranks all members, sums this
 *                                     shard's pairs into the reduce buffers;
 *   evo_get_reduce_buffers            device pointers of grad_sum[ldD] (fp64) and sigma_sum[ldD]
 *                                     (fp32, NULL unless sigma adapts): the caller sums them over
 *                                     the shards in place (all-reduce);
 *   evo_tell_end(s)                   applies the optimiser step from the summed buffers.
 * All shards end with the same centre provided the all-reduce delivers identical bits to all.
 * A solver with shard_pairs == 0 may use the pair too (they then equal evo_tell).
 * Errors: BAD_ORDER (begin without ask, end without begin), INVALID_ARG, CUDA.
 */
evo_status evo_tell_begin(evo_solver* s, const float* d_fitness_all);
evo_status evo_get_reduce_buffers(evo_solver* s, double** d_grad_sum, float** d_sigma_sum, size_t* count);
evo_status evo_tell_end(evo_solver* s);

/* Frees the host handle.  Does not touch the workspace; does not synchronise. */
evo_status evo_destroy(evo_solver* s);

/* ---- helpers -------------------------------------------------------------------------- */

/* Supervised task: bind the batch scored by every member (paper Section 3, supervised tasks
 * provide data and labels).  d_images [batch][28][28] fp32, d_labels [batch] int32 in 0..9;
 * both stay owned by the caller and must outlive the rollouts that use them. */
evo_status evo_set_batch(evo_solver* s, const float* d_images, const int32_t* d_labels);

/* Painting task (paper Section 3, "Concrete and Abstract Painting"): bind the target image,
 * d_target [height][width][3] fp32 in [0,1], owned by the caller, alive during the rollouts.  With
 * this task evo_rollout's d_trace, when given (trace_steps > 0), receives every member's canvas
 * [P][height][width][3].  Errors: INVALID_ARG (NULL), UNSUPPORTED (other task). */
evo_status evo_set_target(evo_solver* s, const float* d_target);

/* Device pointers into the workspace (valid for the solver's lifetime): centre, Adam moments,
 * last gradient (each [ldD] floats, padding zero); ranks [P] int32 and centred-rank weights
 * [P] fp32 of the last tell; eps[H][ldD] of the last ask (NULL in REGENERATED mode). */
evo_status evo_get_center (evo_solver* s, const float** d_center);
evo_status evo_get_moments(evo_solver* s, const float** d_m, const float** d_v);
evo_status evo_get_gradient(evo_solver* s, const float** d_g);
evo_status evo_get_ranks  (evo_solver* s, const int32_t** d_rank, const float** d_u);
evo_status evo_get_eps    (evo_solver* s, const float** d_eps);
/* sigma[ldD] (fp32) in the workspace; evo_set_sigma copies D floats from a device pointer into
 * it, asynchronously on the solver's stream (checkpoint / resume of an adapted sigma). */
evo_status evo_get_sigma  (evo_solver* s, const float** d_sigma);
evo_status evo_set_sigma  (evo_solver* s, const float* d_sigma);

/* Checkpoint / resume: counters are (generation, Adam step).  Both live in device memory and are
 * advanced by the kernel that closes a tell, so evo_ask / evo_rollout / evo_tell pass nothing to
 * their kernels that changes from one generation to the next: a sequence ask -> rollout -> tell
 * captured into a CUDA graph (on the solver's stream, which must not be the legacy default stream)
 * can be replayed, each replay being one more generation.  evo_set_state copies D floats from each
 * non-NULL device pointer into the solver and sets the counters; evo_get_counters reads them back;
 * both therefore synchronise the stream (do not call them while capturing). */
evo_status evo_get_counters(evo_solver* s, uint32_t* generation, uint32_t* adam_step);
evo_status evo_set_state(evo_solver* s, const float* d_center, const float* d_m, const float* d_v,
                         uint32_t generation, uint32_t adam_step);

/* Waits for the solver's stream, returns and clears the device status (EVO_OK,
 * EVO_ERR_NONFINITE, EVO_ERR_TIMEOUT) or EVO_ERR_CUDA if the stream reports a fault. */
evo_status evo_sync_status(evo_solver* s);

/*
 * Checked build only (libevo_debug.so, compiled with -DEVO_DEBUG; the paper has no counterpart: this
 * stands in for a memory checker where none can be run).  In that build every region of the
 * workspace is followed by 256 guard bytes written at evo_create, and the kernels' global stores
 * test their index against the array size, skip the store when it is outside and record the first
 * such site.  evo_debug_check waits for the stream and reports *damaged_region = the index (in
 * layout order) of the first region whose guard bytes changed, or -1; *bounds_site = the first
 * store site that was skipped (0 = none) and *bounds_index = its index.  The normal build returns
 * EVO_ERR_UNSUPPORTED.  Errors: INVALID_ARG (NULL), CUDA.
 */
evo_status evo_debug_check(evo_solver* s, int32_t* damaged_region, uint32_t* bounds_site, uint64_t* bounds_index);

/* Number of kernels the library has launched for this solver so far. */
evo_status evo_launch_count(evo_solver* s, uint64_t* launches);

/*
 * ES gradient without any device allocation (the paper has no counterpart: this entry point
 * exists for deployment reasons only).  It is meant for callers that are not allowed to
 * allocate device memory after start-up and therefore cannot hand evo_create a workspace: a
 * service that distributes all GPU memory once when it boots, or a plug-in inside a host
 * framework whose allocator owns the device.  Computes, like the gradient stage of evo_tell,
 *     d_gradient[d] = (sigma / pop_size) * sum_j (d_u[2j] - d_u[2j+1]) * d_eps[j * ld_eps + d]
 * for d < param_dim, with fp64 partial sums.  d_u[pop_size] (centred-rank weights, fp32),
 * d_eps[pop_size/2][ld_eps] (fp32, ld_eps >= param_dim) and d_gradient[param_dim] are the
 * caller's device buffers; nothing else is needed.
 *   - The split partial sums live in a fixed array of EVO_STATIC_SCRATCH_BYTES that is part of
 *     the library image: every GPU that loads the library carries it until the process ends.
 *     Limit: param_dim rounded up to a multiple of 32 must not exceed
 *     EVO_STATIC_SCRATCH_BYTES / 8 (= 524,288); larger problems return EVO_ERR_WORKSPACE and
 *     must use evo_create / evo_tell with a caller workspace.
 *   - The device that owns the buffers must be current.  The first call on each device looks
 *     up the array's device address (no allocation); make that first call outside of any
 *     stream capture.  No call allocates, frees or synchronises.  The address is cached per
 *     device for the life of the process: do not call again on a device after cudaDeviceReset.
 *   - All calls on a device share the one array, which keeps whatever the previous call left;
 *     each call overwrites every word it reads back, so nothing needs clearing.  Two calls
 *     whose kernels may overlap on the GPU (different streams, or the same stream from two
 *     threads) race on it: serialise them.
 * Errors: INVALID_ARG (NULL pointer, odd or zero pop_size, ld_eps < param_dim), WORKSPACE
 * (param_dim beyond the limit), CUDA (address lookup or launch failed).
 */
#define EVO_STATIC_SCRATCH_BYTES (4u << 20)
evo_status evo_es_gradient_static(const float* d_u, const float* d_eps, uint32_t pop_size,
                                  uint32_t param_dim, size_t ld_eps, float sigma,
                                  float* d_gradient, void* cuda_stream);

const char* evo_status_string(evo_status st);
uint32_t    evo_version(void);            /* major*10000 + minor*100 + patch: 1.1.0 = 10100 */

#ifdef __cplusplus
}
#endif
#endif /* EVO_H */
