// Host side of the C-ABI declared in include/evo.h: argument checks, workspace layout and
// kernel launches.  No device memory is allocated here; nothing synchronises except
// evo_sync_status / evo_get_counters.
#include "internal.h"

#include <cmath>
#include <cstring>
#include <new>

using namespace evo;

struct evo_solver {
    evo_config   cfg;
    Layout       lay;
    char*        ws;
    cudaStream_t stream;
    uint32_t     generation;
    bool         asked;            // an ask without a matching tell is outstanding
    bool         telling;          // evo_tell_begin done, evo_tell_end outstanding
    uint32_t     local_pop;        // members this solver samples and evaluates (the shard's)
    uint32_t     pair0;            // first global pair of the shard
    bool         ever_asked;
    const float*   d_images;
    const int32_t* d_labels;
    const float*   d_target;
    uint64_t     launches;
    uint32_t     k0, k1;
    bool         rollout_prepared;  // per-kernel attributes are set by the solver's first roll-out only
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
constexpr int kCanaryByte = 0xA5;

static evo_status check_config(const evo_config* c)
{
    if (!c || c->struct_size != sizeof(evo_config)) return EVO_ERR_INVALID_ARG;
    if (c->pop_size < 2 || (c->pop_size & 1u) || c->param_dim < 1) return EVO_ERR_INVALID_ARG;
    if (c->param_dim > kMaxParamDim) return EVO_ERR_INVALID_ARG;      // the row pitch must fit 32 bits
    if (!(c->sigma > 0.f) || !std::isfinite(c->sigma) || !std::isfinite(c->lr)) return EVO_ERR_INVALID_ARG;
    if (c->noise_mode > EVO_NOISE_REGENERATED) return EVO_ERR_INVALID_ARG;
    if (c->beta1 < 0.f || c->beta1 >= 1.f || c->beta2 < 0.f || c->beta2 >= 1.f || c->adam_eps < 0.f)
        return EVO_ERR_INVALID_ARG;
    if (c->rollout_kernel > EVO_ROLLOUT_TILED) return EVO_ERR_INVALID_ARG;
    if (c->optimizer > EVO_OPT_CLIPUP || c->sigma_mode > EVO_SIGMA_PGPE) return EVO_ERR_INVALID_ARG;
    if (c->clipup_momentum < 0.f || c->clipup_momentum >= 1.f || c->clipup_max_speed < 0.f) return EVO_ERR_INVALID_ARG;
    if (c->sigma_lr < 0.f || c->sigma_max_change < 0.f || c->sigma_max_change >= 1.f) return EVO_ERR_INVALID_ARG;
    if (c->wait_cycles_log2 != 0 && (c->wait_cycles_log2 < 10 || c->wait_cycles_log2 > 40)) return EVO_ERR_INVALID_ARG;
    if (c->debug_flags & ~static_cast<uint32_t>(EVO_DEBUG_DROP_COMPLETION)) return EVO_ERR_INVALID_ARG;
    if (c->shard_pairs > 0 &&
        (c->shard_first_pair >= c->pop_size / 2u || c->shard_pairs > c->pop_size / 2u - c->shard_first_pair))
        return EVO_ERR_INVALID_ARG;
    switch (c->task_kind) {
        case EVO_TASK_NONE: break;
        case EVO_TASK_CARTPOLE:
        case EVO_TASK_TANH_LINEAR:
            if (c->policy_kind != EVO_POLICY_MLP) return EVO_ERR_INVALID_ARG;
            if (c->episodes < 1 || c->horizon < 1) return EVO_ERR_INVALID_ARG;
            if (c->trace_steps > c->horizon) return EVO_ERR_INVALID_ARG;   // the trace pitch is trace_steps
            if (!rollout_mlp_supported(*c)) return EVO_ERR_INVALID_ARG;
            if (c->task_kind == EVO_TASK_CARTPOLE) {
                const float* tp = c->task_param;
                if (!(tp[EVO_CP_CART_MASS] > 0.f) || !(tp[EVO_CP_POLE_MASS] > 0.f) ||
                    !(tp[EVO_CP_POLE_HALF_LENGTH] > 0.f) || !(tp[EVO_CP_DT] > 0.f) ||
                    !(tp[EVO_CP_INIT_RANGE] >= 0.f))
                    return EVO_ERR_INVALID_ARG;
            }
            break;
        case EVO_TASK_SUPERVISED:
            if (c->policy_kind != EVO_POLICY_CNN_28 || c->param_dim != kCnnParams || c->batch < 1)
                return EVO_ERR_INVALID_ARG;
            break;
        case EVO_TASK_SEQ2SEQ_ADD: {
            const float nd = c->task_param[EVO_S2S_DIGITS];
            if (c->policy_kind != EVO_POLICY_LSTM_SEQ2SEQ || !(nd >= 1.f) || nd != static_cast<float>(static_cast<uint32_t>(nd)))
                return EVO_ERR_INVALID_ARG;
            if (!s2s_supported(c->layer_sizes[0], static_cast<uint32_t>(nd), c->batch) ||
                c->param_dim != s2s_param_count(c->layer_sizes[0]))
                return EVO_ERR_INVALID_ARG;
            break;
        }
        case EVO_TASK_PAINT: {
            const float w = c->task_param[EVO_PAINT_WIDTH], h = c->task_param[EVO_PAINT_HEIGHT];
            const float bg = c->task_param[EVO_PAINT_BACKGROUND];
            if (c->policy_kind != EVO_POLICY_NONE || !(w >= 1.f) || !(h >= 1.f) || !(w <= 4096.f) || !(h <= 4096.f) ||
                w != static_cast<float>(static_cast<uint32_t>(w)) || h != static_cast<float>(static_cast<uint32_t>(h)) ||
                !(bg >= 0.f) || !(bg <= 1.f))
                return EVO_ERR_INVALID_ARG;
            if (!paint_supported(c->param_dim, static_cast<uint32_t>(w), static_cast<uint32_t>(h))) return EVO_ERR_INVALID_ARG;
            break;
        }
        default: return EVO_ERR_INVALID_ARG;
    }
    return EVO_OK;
}

static evo_status make_layout(const evo_config& c, Layout* L)
{
    const size_t P = c.pop_size;                                        // global population (ranks)
    const size_t Pl = c.shard_pairs ? 2u * c.shard_pairs : c.pop_size;   // members sampled / evaluated here
    const size_t Hl = Pl / 2;
    const uint32_t ldD = static_cast<uint32_t>(align_up(c.param_dim, 32));
    L->ldD = ldD;
    L->grad_splits = gradient_splits(static_cast<uint32_t>(Hl), ldD);
    L->EB = 1; L->n_eb = 1;
    if (c.task_kind == EVO_TASK_CARTPOLE || c.task_kind == EVO_TASK_TANH_LINEAR)
        rollout_mlp_plan(c, &L->EB, &L->n_eb);
    size_t off = 0;
    L->n_canaries = 0;
    // every region starts 256-byte aligned; the checked build puts kCanaryBytes of guard words behind each
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 256);
        if (kCanaryBytes && L->n_canaries < kMaxRegions) { L->canary[L->n_canaries++] = off; off += kCanaryBytes; }
        return o;
    };
    const size_t row = static_cast<size_t>(ldD) * sizeof(float);
    L->status = take(sizeof(DeviceStatus));
    L->center = take(row);
    L->m = take(row);
    L->v = take(row);
    L->g = take(row);
    L->sigma = take(row);
    L->u = take(P * sizeof(float));
    L->rank = take(P * sizeof(int32_t));
    L->grad_partial = take(2 * row * L->grad_splits);          // fp64 partial sums
    L->sigma_partial = take(c.sigma_mode == EVO_SIGMA_PGPE ? row * L->grad_splits : 0);
    L->grad_sum = take(2 * row);                                // fp64, summed over shards by the caller
    L->sigma_sum = take(c.sigma_mode == EVO_SIGMA_PGPE ? row : 0);
    L->norms = take(clipup_norm_doubles(ldD) * sizeof(double));
    L->fit_partial = take(Pl * L->n_eb * sizeof(float));
    L->task_const = take(kTlNx * (kTlNx + kTlNa) * sizeof(float));
    size_t cnn = 0;
    if (c.task_kind == EVO_TASK_SUPERVISED) {
        cnn = cnn_scratch_bytes(static_cast<uint32_t>(Pl), c.batch);
        const size_t tc = cnn_tc_scratch_bytes(static_cast<uint32_t>(Pl), c.batch);
        if (tc > cnn) cnn = tc;
    }
    if (c.task_kind == EVO_TASK_SEQ2SEQ_ADD) cnn = s2s_scratch_bytes(static_cast<uint32_t>(Pl), c.batch);
    if (c.task_kind == EVO_TASK_PAINT)
        cnn = paint_scratch_bytes(static_cast<uint32_t>(Pl), static_cast<uint32_t>(c.task_param[EVO_PAINT_WIDTH]),
                                  static_cast<uint32_t>(c.task_param[EVO_PAINT_HEIGHT]));
    L->cnn_scratch = take(cnn);                                 // scratch of the single-step tasks
    L->theta = take(row * Pl);
    L->eps = take(c.noise_mode == EVO_NOISE_STORED ? row * Hl : 0);
    L->total = off;
    return EVO_OK;
}

extern "C" {

evo_status evo_workspace_bytes(const evo_config* cfg, size_t* bytes)
{
    if (!bytes) return EVO_ERR_INVALID_ARG;
    evo_status st = check_config(cfg);
    if (st != EVO_OK) return st;
    Layout L;
    make_layout(*cfg, &L);
    *bytes = L.total;
    return EVO_OK;
}

evo_status evo_create(const evo_config* cfg_in, void* d_workspace, size_t workspace_bytes,
                      void* cuda_stream, evo_solver** out)
{
    if (!out) return EVO_ERR_INVALID_ARG;
    *out = nullptr;
    evo_status st = check_config(cfg_in);
    if (st != EVO_OK) return st;
    if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return EVO_ERR_INVALID_ARG;
    evo_solver* s = new (std::nothrow) evo_solver();
    if (!s) return EVO_ERR_INVALID_ARG;
    s->cfg = *cfg_in;
    if (s->cfg.beta1 == 0.f) s->cfg.beta1 = 0.9f;
    if (s->cfg.beta2 == 0.f) s->cfg.beta2 = 0.999f;
    if (s->cfg.adam_eps == 0.f) s->cfg.adam_eps = 1e-8f;
    if (s->cfg.clipup_momentum == 0.f) s->cfg.clipup_momentum = 0.9f;
    if (s->cfg.clipup_max_speed == 0.f) s->cfg.clipup_max_speed = 2.f * s->cfg.lr;
    if (s->cfg.sigma_lr == 0.f) s->cfg.sigma_lr = 0.1f;
    if (s->cfg.sigma_max_change == 0.f) s->cfg.sigma_max_change = 0.2f;
    if (s->cfg.wait_cycles_log2 == 0) s->cfg.wait_cycles_log2 = 31;       // ~1 s at 2 GHz
    make_layout(s->cfg, &s->lay);
    if (workspace_bytes < s->lay.total) { delete s; return EVO_ERR_WORKSPACE; }
    s->ws = static_cast<char*>(d_workspace);
    s->stream = static_cast<cudaStream_t>(cuda_stream);
    s->generation = 0;
    s->asked = false;
    s->telling = false;
    s->local_pop = s->cfg.shard_pairs ? 2u * s->cfg.shard_pairs : s->cfg.pop_size;
    s->pair0 = s->cfg.shard_pairs ? s->cfg.shard_first_pair : 0u;
    s->ever_asked = false;
    s->d_images = nullptr;
    s->d_labels = nullptr;
    s->d_target = nullptr;
    s->launches = 0;
    s->rollout_prepared = false;
    s->k0 = static_cast<uint32_t>(s->cfg.seed & 0xFFFFFFFFull);
    s->k1 = static_cast<uint32_t>(s->cfg.seed >> 32);
    const Layout& L = s->lay;
    int n = launch_init(s->stream, reinterpret_cast<float*>(s->ws + L.center),
                        reinterpret_cast<float*>(s->ws + L.m), reinterpret_cast<float*>(s->ws + L.v),
                        reinterpret_cast<float*>(s->ws + L.g), reinterpret_cast<float*>(s->ws + L.sigma),
                        s->cfg.sigma, s->cfg.param_dim, L.ldD,
                        reinterpret_cast<DeviceStatus*>(s->ws + L.status), s->cfg.wait_cycles_log2,
                        s->cfg.debug_flags);
    if (n < 0) { delete s; return EVO_ERR_CUDA; }
    s->launches += n;
    n = launch_task_constants(s->stream, s->cfg.task_kind, s->k0, s->k1,
                              reinterpret_cast<float*>(s->ws + L.task_const));
    if (n < 0) { delete s; return EVO_ERR_CUDA; }
    s->launches += n;
    for (int i = 0; i < L.n_canaries; ++i)          // checked build only (n_canaries is 0 otherwise)
        if (cudaMemsetAsync(s->ws + L.canary[i], kCanaryByte, kCanaryBytes, s->stream) != cudaSuccess) {
            delete s;
            return EVO_ERR_CUDA;
        }
    *out = s;
    return EVO_OK;
}

evo_status evo_ask(evo_solver* s, const float** d_theta, size_t* ld_theta)
{
    if (!s) return EVO_ERR_INVALID_ARG;
    const Layout& L = s->lay;
    float* theta = reinterpret_cast<float*>(s->ws + L.theta);
    float* eps = s->cfg.noise_mode == EVO_NOISE_STORED ? reinterpret_cast<float*>(s->ws + L.eps) : nullptr;
    const int n = launch_ask(s->stream, reinterpret_cast<const float*>(s->ws + L.center),
                             reinterpret_cast<const float*>(s->ws + L.sigma),
                             s->k0, s->k1, reinterpret_cast<const DeviceStatus*>(s->ws + L.status), s->pair0, s->local_pop / 2, s->cfg.param_dim, L.ldD,
                             theta, eps);
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    s->asked = true;
    s->ever_asked = true;
    if (d_theta) *d_theta = theta;
    if (ld_theta) *ld_theta = L.ldD;
    return EVO_OK;
}

evo_status evo_set_batch(evo_solver* s, const float* d_images, const int32_t* d_labels)
{
    if (!s || !d_images || !d_labels) return EVO_ERR_INVALID_ARG;
    if (s->cfg.task_kind != EVO_TASK_SUPERVISED) return EVO_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(d_images) & 15u) return EVO_ERR_INVALID_ARG;
    s->d_images = d_images;
    s->d_labels = d_labels;
    return EVO_OK;
}

evo_status evo_set_target(evo_solver* s, const float* d_target)
{
    if (!s || !d_target) return EVO_ERR_INVALID_ARG;
    if (s->cfg.task_kind != EVO_TASK_PAINT) return EVO_ERR_UNSUPPORTED;
    s->d_target = d_target;
    return EVO_OK;
}

evo_status evo_rollout(evo_solver* s, const float* d_theta, float* d_fitness, float* d_trace)
{
    if (!s || !d_fitness) return EVO_ERR_INVALID_ARG;
    const evo_config& c = s->cfg;
    const Layout& L = s->lay;
    if (c.task_kind == EVO_TASK_NONE) return EVO_ERR_UNSUPPORTED;
    if (!d_theta) {
        if (!s->ever_asked) return EVO_ERR_BAD_ORDER;
        d_theta = reinterpret_cast<const float*>(s->ws + L.theta);
    } else if (reinterpret_cast<uintptr_t>(d_theta) & 15u) {
        return EVO_ERR_INVALID_ARG;
    }
    if (c.task_kind == EVO_TASK_SUPERVISED) {
        if (!s->d_images) return EVO_ERR_BAD_ORDER;
        if (d_trace) return EVO_ERR_UNSUPPORTED;
        // GENERIC selects the CUDA-core kernel, anything else the tensor-core path
        const int n = c.rollout_kernel == EVO_ROLLOUT_GENERIC
            ? launch_rollout_cnn(s->stream, d_theta, L.ldD, s->local_pop, s->d_images, s->d_labels, c.batch,
                                 s->ws + L.cnn_scratch, d_fitness)
            : launch_rollout_cnn_tc(s->stream, d_theta, L.ldD, s->local_pop, s->d_images, s->d_labels, c.batch,
                                    s->ws + L.cnn_scratch, d_fitness,
                                    reinterpret_cast<DeviceStatus*>(s->ws + L.status));
        if (n < 0) return n == -2 ? EVO_ERR_UNSUPPORTED : EVO_ERR_CUDA;
        s->launches += n;
        return EVO_OK;
    }
    if (d_trace && c.trace_steps == 0) return EVO_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_trace) & 15u) return EVO_ERR_INVALID_ARG;   // written with 128-bit stores
    if (c.task_kind == EVO_TASK_PAINT) {
        if (!s->d_target) return EVO_ERR_BAD_ORDER;
        const int n = launch_rollout_paint(s->stream, d_theta, L.ldD, s->local_pop, c.param_dim,
                                           static_cast<uint32_t>(c.task_param[EVO_PAINT_WIDTH]),
                                           static_cast<uint32_t>(c.task_param[EVO_PAINT_HEIGHT]),
                                           c.task_param[EVO_PAINT_BACKGROUND], s->d_target, s->ws + L.cnn_scratch,
                                           d_fitness, d_trace);
        if (n < 0) return EVO_ERR_CUDA;
        s->launches += n;
        return EVO_OK;
    }
    if (c.task_kind == EVO_TASK_SEQ2SEQ_ADD) {
        // d_trace, when given, receives the logits [P][batch][digits+1][12] (CUDA-core kernel)
        const int n = launch_rollout_s2s(s->stream, d_theta, L.ldD, s->local_pop, c.layer_sizes[0],
                                         static_cast<uint32_t>(c.task_param[EVO_S2S_DIGITS]), c.batch, s->k0, s->k1,
                                         c.rollout_kernel, s->ws + L.cnn_scratch, d_fitness, d_trace,
                                         reinterpret_cast<DeviceStatus*>(s->ws + L.status));
        if (n < 0) return n == -2 ? EVO_ERR_UNSUPPORTED : EVO_ERR_CUDA;
        s->launches += n;
        return EVO_OK;
    }
    RolloutMlpArgs a;
    std::memset(&a, 0, sizeof(a));
    a.theta = d_theta;
    a.fit_partial = reinterpret_cast<float*>(s->ws + L.fit_partial);
    a.trace = d_trace;
    a.task_const = reinterpret_cast<const float*>(s->ws + L.task_const);
    a.P = s->local_pop;
    a.ldD = L.ldD;
    a.n_layers = c.n_layers;
    a.max_width = 0;
    for (uint32_t l = 0; l <= c.n_layers; ++l) {
        a.sizes[l] = c.layer_sizes[l];
        if (c.layer_sizes[l] > a.max_width) a.max_width = c.layer_sizes[l];
    }
    a.action_scale = c.action_scale;
    a.task = c.task_kind;
    a.E = c.episodes; a.T = c.horizon; a.EB = L.EB; a.n_eb = L.n_eb;
    a.trace_T = c.trace_steps < c.horizon ? c.trace_steps : c.horizon;
    a.k0 = s->k0; a.k1 = s->k1;
    std::memcpy(a.tp, c.task_param, sizeof(a.tp));
    a.attr_done = s->rollout_prepared ? 1u : 0u;
    const int n = launch_rollout_mlp(s->stream, a, c.rollout_kernel, d_fitness,
                                     reinterpret_cast<DeviceStatus*>(s->ws + L.status));
    if (n < 0) return n == -2 ? EVO_ERR_UNSUPPORTED : EVO_ERR_CUDA;
    s->rollout_prepared = true;
    s->launches += n;
    return EVO_OK;
}

static TellArgs tell_args(evo_solver* s)
{
    const evo_config& c = s->cfg;
    const Layout& L = s->lay;
    TellArgs t;
    t.u = reinterpret_cast<const float*>(s->ws + L.u);
    t.eps = c.noise_mode == EVO_NOISE_STORED ? reinterpret_cast<const float*>(s->ws + L.eps) : nullptr;
    t.k0 = s->k0; t.k1 = s->k1;
    t.H = s->local_pop / 2; t.D = c.param_dim; t.ldD = L.ldD; t.splits = L.grad_splits;
    t.pair0 = s->pair0; t.P = c.pop_size;
    t.partial = reinterpret_cast<double*>(s->ws + L.grad_partial);
    t.sigma_partial = c.sigma_mode == EVO_SIGMA_PGPE ? reinterpret_cast<float*>(s->ws + L.sigma_partial) : nullptr;
    t.norms = reinterpret_cast<double*>(s->ws + L.norms);
    t.sigma_vec = reinterpret_cast<float*>(s->ws + L.sigma);
    t.lr = c.lr; t.beta1 = c.beta1; t.beta2 = c.beta2; t.adam_eps = c.adam_eps;
    t.optimizer = c.optimizer; t.clipup_momentum = c.clipup_momentum; t.clipup_max_speed = c.clipup_max_speed;
    t.sigma_lr = c.sigma_lr; t.sigma_max_change = c.sigma_max_change;
    t.center = reinterpret_cast<float*>(s->ws + L.center);
    t.m = reinterpret_cast<float*>(s->ws + L.m);
    t.v = reinterpret_cast<float*>(s->ws + L.v);
    t.g = reinterpret_cast<float*>(s->ws + L.g);
    t.status = reinterpret_cast<DeviceStatus*>(s->ws + L.status);
    return t;
}

evo_status evo_tell(evo_solver* s, const float* d_fitness)
{
    if (!s || !d_fitness) return EVO_ERR_INVALID_ARG;
    if (s->cfg.shard_pairs) return EVO_ERR_UNSUPPORTED;        // a shard needs the exchange in between
    if (!s->asked || s->telling) return EVO_ERR_BAD_ORDER;
    const Layout& L = s->lay;
    const TellArgs t = tell_args(s);
    int n = launch_rank(s->stream, d_fitness, s->cfg.pop_size, reinterpret_cast<int32_t*>(s->ws + L.rank),
                        reinterpret_cast<float*>(s->ws + L.u), t.status);
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    n = launch_gradient_update(s->stream, t);
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    s->asked = false;
    s->generation += 1;
    return EVO_OK;
}

evo_status evo_tell_begin(evo_solver* s, const float* d_fitness_all)
{
    if (!s || !d_fitness_all) return EVO_ERR_INVALID_ARG;
    if (!s->asked || s->telling) return EVO_ERR_BAD_ORDER;
    const Layout& L = s->lay;
    const TellArgs t = tell_args(s);
    int n = launch_rank(s->stream, d_fitness_all, s->cfg.pop_size, reinterpret_cast<int32_t*>(s->ws + L.rank),
                        reinterpret_cast<float*>(s->ws + L.u), t.status);
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    n = launch_gradient_sums(s->stream, t, reinterpret_cast<double*>(s->ws + L.grad_sum),
                             reinterpret_cast<float*>(s->ws + L.sigma_sum));
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    s->telling = true;
    return EVO_OK;
}

evo_status evo_get_reduce_buffers(evo_solver* s, double** d_grad_sum, float** d_sigma_sum, size_t* count)
{
    if (!s || !d_grad_sum || !d_sigma_sum || !count) return EVO_ERR_INVALID_ARG;
    *d_grad_sum = reinterpret_cast<double*>(s->ws + s->lay.grad_sum);
    *d_sigma_sum = s->cfg.sigma_mode == EVO_SIGMA_PGPE ? reinterpret_cast<float*>(s->ws + s->lay.sigma_sum) : nullptr;
    *count = s->lay.ldD;
    return EVO_OK;
}

evo_status evo_tell_end(evo_solver* s)
{
    if (!s) return EVO_ERR_INVALID_ARG;
    if (!s->telling) return EVO_ERR_BAD_ORDER;
    const Layout& L = s->lay;
    const TellArgs t = tell_args(s);
    const int n = launch_update_from_sums(s->stream, t, reinterpret_cast<const double*>(s->ws + L.grad_sum),
                                          reinterpret_cast<const float*>(s->ws + L.sigma_sum));
    if (n < 0) return EVO_ERR_CUDA;
    s->launches += n;
    s->telling = false;
    s->asked = false;
    s->generation += 1;
    return EVO_OK;
}

evo_status evo_destroy(evo_solver* s)
{
    if (!s) return EVO_ERR_INVALID_ARG;
    delete s;
    return EVO_OK;
}

evo_status evo_get_center(evo_solver* s, const float** d_center)
{
    if (!s || !d_center) return EVO_ERR_INVALID_ARG;
    *d_center = reinterpret_cast<const float*>(s->ws + s->lay.center);
    return EVO_OK;
}

evo_status evo_get_moments(evo_solver* s, const float** d_m, const float** d_v)
{
    if (!s || !d_m || !d_v) return EVO_ERR_INVALID_ARG;
    *d_m = reinterpret_cast<const float*>(s->ws + s->lay.m);
    *d_v = reinterpret_cast<const float*>(s->ws + s->lay.v);
    return EVO_OK;
}

evo_status evo_get_gradient(evo_solver* s, const float** d_g)
{
    if (!s || !d_g) return EVO_ERR_INVALID_ARG;
    *d_g = reinterpret_cast<const float*>(s->ws + s->lay.g);
    return EVO_OK;
}

evo_status evo_get_ranks(evo_solver* s, const int32_t** d_rank, const float** d_u)
{
    if (!s || !d_rank || !d_u) return EVO_ERR_INVALID_ARG;
    *d_rank = reinterpret_cast<const int32_t*>(s->ws + s->lay.rank);
    *d_u = reinterpret_cast<const float*>(s->ws + s->lay.u);
    return EVO_OK;
}

evo_status evo_get_eps(evo_solver* s, const float** d_eps)
{
    if (!s || !d_eps) return EVO_ERR_INVALID_ARG;
    *d_eps = s->cfg.noise_mode == EVO_NOISE_STORED ? reinterpret_cast<const float*>(s->ws + s->lay.eps)
                                                   : nullptr;
    return EVO_OK;
}

evo_status evo_get_sigma(evo_solver* s, const float** d_sigma)
{
    if (!s || !d_sigma) return EVO_ERR_INVALID_ARG;
    *d_sigma = reinterpret_cast<const float*>(s->ws + s->lay.sigma);
    return EVO_OK;
}

evo_status evo_set_sigma(evo_solver* s, const float* d_sigma)
{
    if (!s || !d_sigma) return EVO_ERR_INVALID_ARG;
    const size_t bytes = static_cast<size_t>(s->cfg.param_dim) * sizeof(float);
    if (cudaMemcpyAsync(s->ws + s->lay.sigma, d_sigma, bytes, cudaMemcpyDeviceToDevice, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    return EVO_OK;
}

evo_status evo_get_counters(evo_solver* s, uint32_t* generation, uint32_t* adam_step)
{
    if (!s || !generation || !adam_step) return EVO_ERR_INVALID_ARG;
    DeviceStatus h;
    if (cudaMemcpyAsync(&h, s->ws + s->lay.status, sizeof(h), cudaMemcpyDeviceToHost, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    if (cudaStreamSynchronize(s->stream) != cudaSuccess) return EVO_ERR_CUDA;
    *generation = h.generation;
    *adam_step = h.adam_step;
    s->generation = h.generation;                 // host mirror (informative only)
    return EVO_OK;
}

evo_status evo_set_state(evo_solver* s, const float* d_center, const float* d_m, const float* d_v,
                         uint32_t generation, uint32_t adam_step)
{
    if (!s) return EVO_ERR_INVALID_ARG;
    const size_t bytes = static_cast<size_t>(s->cfg.param_dim) * sizeof(float);
    const Layout& L = s->lay;
    if (d_center && cudaMemcpyAsync(s->ws + L.center, d_center, bytes, cudaMemcpyDeviceToDevice, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    if (d_m && cudaMemcpyAsync(s->ws + L.m, d_m, bytes, cudaMemcpyDeviceToDevice, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    if (d_v && cudaMemcpyAsync(s->ws + L.v, d_v, bytes, cudaMemcpyDeviceToDevice, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    static_assert(offsetof(DeviceStatus, generation) == offsetof(DeviceStatus, adam_step) + sizeof(uint32_t), "adjacent counters");
    const uint32_t counters[2] = { adam_step, generation };
    if (cudaMemcpyAsync(s->ws + L.status + offsetof(DeviceStatus, adam_step), counters, sizeof(counters),
                        cudaMemcpyHostToDevice, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    if (cudaStreamSynchronize(s->stream) != cudaSuccess) return EVO_ERR_CUDA;   // the counters are a stack value
    s->generation = generation;
    s->asked = false;
    s->telling = false;
    return EVO_OK;
}

evo_status evo_sync_status(evo_solver* s)
{
    if (!s) return EVO_ERR_INVALID_ARG;
    DeviceStatus h;
    if (cudaMemcpyAsync(&h, s->ws + s->lay.status, sizeof(h), cudaMemcpyDeviceToHost, s->stream) != cudaSuccess)
        return EVO_ERR_CUDA;
    if (cudaStreamSynchronize(s->stream) != cudaSuccess) return EVO_ERR_CUDA;
    if (h.sticky) {
        const uint32_t zero = 0;
        if (cudaMemcpyAsync(s->ws + s->lay.status + offsetof(DeviceStatus, sticky), &zero, sizeof(zero),
                            cudaMemcpyHostToDevice, s->stream) != cudaSuccess)
            return EVO_ERR_CUDA;
        if (cudaStreamSynchronize(s->stream) != cudaSuccess) return EVO_ERR_CUDA;
        if (h.sticky & (1u << EVO_ERR_TIMEOUT)) return EVO_ERR_TIMEOUT;
        if (h.sticky & (1u << EVO_ERR_NONFINITE)) return EVO_ERR_NONFINITE;
        return EVO_ERR_CUDA;
    }
    return EVO_OK;
}

evo_status evo_debug_check(evo_solver* s, int32_t* damaged_region, uint32_t* bounds_site, uint64_t* bounds_index)
{
    if (!s || !damaged_region || !bounds_site || !bounds_index) return EVO_ERR_INVALID_ARG;
#ifdef EVO_DEBUG
    *damaged_region = -1; *bounds_site = 0; *bounds_index = 0;
    if (cudaStreamSynchronize(s->stream) != cudaSuccess) return EVO_ERR_CUDA;
    unsigned char guard[kCanaryBytes];
    for (int i = 0; i < s->lay.n_canaries && *damaged_region < 0; ++i) {
        if (cudaMemcpy(guard, s->ws + s->lay.canary[i], kCanaryBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
            return EVO_ERR_CUDA;
        for (size_t b = 0; b < kCanaryBytes; ++b)
            if (guard[b] != kCanaryByte) { *damaged_region = i; break; }
    }
    DeviceStatus h;
    if (cudaMemcpy(&h, s->ws + s->lay.status, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return EVO_ERR_CUDA;
    *bounds_site = h.bounds_site;
    *bounds_index = (static_cast<uint64_t>(h.bounds_index_hi) << 32) | h.bounds_index_lo;
    return EVO_OK;
#else
    return EVO_ERR_UNSUPPORTED;
#endif
}

evo_status evo_launch_count(evo_solver* s, uint64_t* launches)
{
    if (!s || !launches) return EVO_ERR_INVALID_ARG;
    *launches = s->launches;
    return EVO_OK;
}

const char* evo_status_string(evo_status st)
{
    switch (st) {
        case EVO_OK: return "ok";
        case EVO_ERR_INVALID_ARG: return "invalid argument";
        case EVO_ERR_BAD_ORDER: return "call out of order";
        case EVO_ERR_WORKSPACE: return "workspace too small";
        case EVO_ERR_CUDA: return "CUDA error";
        case EVO_ERR_NONFINITE: return "non-finite fitness, update skipped";
        case EVO_ERR_TIMEOUT: return "device-side wait timed out";
        case EVO_ERR_UNSUPPORTED: return "unsupported configuration";
    }
    return "unknown status";
}

uint32_t evo_version(void) { return 10100; }   // 1.1.0

}  // extern "C"
