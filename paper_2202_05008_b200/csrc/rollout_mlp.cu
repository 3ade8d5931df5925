// Fused control-task rollout: one kernel runs all T steps of policy + task for a block of
// episodes of one population member.  The member's MLP weights are read from HBM once and stay
// in shared memory for the whole roll-out; task state lives in registers / shared memory and is
// never written to HBM (except the optional debug trace).  Paper Section 2 (simulation manager:
// roll-out loop, central roll-out seeds), Section 4 (PolicyNetwork.get_actions over the whole
// population with parameters as data; VectorizedTask.reset/step; identical initial observations
// for every member).
//
//   k_rollout_mlp_generic   any layer count / widths (runtime), the reference device path
//   k_rollout_mlp_tiled<..> compile-time shapes with register-tiled layers (the fast path)
#include "internal.h"
#include "noise.cuh"
#include "tasks.cuh"

namespace evo {

// ------------------------------------------------------------------------------------------
// generic kernel: block = (member, episode block); 128 threads; activations in shared memory
// laid out [unit][episode]; every thread owns (unit, episode) items of each layer in turn.
// ------------------------------------------------------------------------------------------
constexpr int kGenericThreads = 128;

__global__ void __launch_bounds__(kGenericThreads)
k_rollout_mlp_generic(const RolloutMlpArgs a, const DeviceStatus* __restrict__ status)
{
    extern __shared__ __align__(16) float smem[];
    const uint32_t member = blockIdx.x, eb = blockIdx.y;
    const uint32_t e0 = eb * a.EB;
    const uint32_t nE = min(a.EB, a.E - e0);          // episodes of this block
    const uint32_t EB = a.EB;
    const uint32_t tid = threadIdx.x;
    const PhiloxKey key = philox_key(a.k0, a.k1);
    const uint32_t generation = status->generation;

    uint32_t n_params = 0;
    for (uint32_t l = 0; l < a.n_layers; ++l) n_params += a.sizes[l + 1] * a.sizes[l] + a.sizes[l + 1];
    const uint32_t n_in0 = a.sizes[0], n_act = a.sizes[a.n_layers];

    float* sp = smem;
    float* buf0 = sp; sp += a.max_width * EB;
    float* buf1 = sp; sp += a.max_width * EB;
    float* obs  = sp; sp += n_in0 * EB;
    float* act  = sp; sp += n_act * EB;
    float* nxt  = sp; sp += (a.task == EVO_TASK_TANH_LINEAR ? kTlNx * EB : 0);
    float* tcon = sp; sp += (a.task == EVO_TASK_TANH_LINEAR ? kTlNx * (kTlNx + kTlNa) : 0);
    float* rets = sp; sp += EB;
    float* wsm  = sp;

    const float* wrow = a.theta + static_cast<size_t>(member) * a.ldD;
    const float* w = wrow;
    if (a.weights_in_smem) {
        for (uint32_t i = tid; i < n_params; i += blockDim.x) wsm[i] = wrow[i];
        w = wsm;
    }
    if (a.task == EVO_TASK_TANH_LINEAR)
        for (uint32_t i = tid; i < kTlNx * (kTlNx + kTlNa); i += blockDim.x) tcon[i] = a.task_const[i];

    // ---- reset -------------------------------------------------------------------------
    CartpoleConst cpc{};
    CpState cps{};
    float ret = 0.f;
    if (a.task == EVO_TASK_CARTPOLE) {
        cpc = cartpole_const(a.tp);
        if (tid < nE) {
            cps = cartpole_reset(key, generation, e0 + tid, a.tp[EVO_CP_INIT_RANGE]);
            float sn, cs;
            sincosf(cps.th, &sn, &cs);
            obs[0 * EB + tid] = cps.x;  obs[1 * EB + tid] = cps.xd;
            obs[2 * EB + tid] = cs;     obs[3 * EB + tid] = sn;
            obs[4 * EB + tid] = cps.thd;
        }
    } else {
        for (uint32_t item = tid; item < (kTlNx / 4) * nE; item += blockDim.x) {
            const uint32_t q = item / nE, e = item % nE;
            const float4 z = stream_normal4(key, 1u, generation, e0 + e, q);
            obs[(4 * q + 0) * EB + e] = z.x; obs[(4 * q + 1) * EB + e] = z.y;
            obs[(4 * q + 2) * EB + e] = z.z; obs[(4 * q + 3) * EB + e] = z.w;
        }
    }
    __syncthreads();

    // ---- time loop -----------------------------------------------------------------------
    for (uint32_t t = 0; t < a.T; ++t) {
        const float* in = obs;
        const float* lw = w;
        for (uint32_t l = 0; l < a.n_layers; ++l) {
            const uint32_t n_in = a.sizes[l], n_out = a.sizes[l + 1];
            const bool last = (l + 1 == a.n_layers);
            float* out = last ? act : ((l & 1u) ? buf1 : buf0);
            const float* bias = lw + n_out * n_in;
            for (uint32_t item = tid; item < n_out * nE; item += blockDim.x) {
                const uint32_t i = item / nE, e = item % nE;
                const float* wr = lw + i * n_in;
                float acc = bias[i];
                for (uint32_t k = 0; k < n_in; ++k) acc = fmaf(wr[k], in[k * EB + e], acc);
                const float y = tanhf(acc);
                out[i * EB + e] = last ? a.action_scale * y : y;
            }
            __syncthreads();
            in = out;
            lw += n_out * n_in + n_out;
        }

        if (a.task == EVO_TASK_CARTPOLE) {
            if (tid < nE) {
                cps = cartpole_step(cpc, cps, act[tid]);
                float sn, cs;
                sincosf(cps.th, &sn, &cs);
                ret += cs * expf(-cps.x * cps.x);            // reward on the post-step state
                obs[0 * EB + tid] = cps.x;  obs[1 * EB + tid] = cps.xd;
                obs[2 * EB + tid] = cs;     obs[3 * EB + tid] = sn;
                obs[4 * EB + tid] = cps.thd;
                if (a.trace && t < a.trace_T) {
                    float* tr = a.trace + ((static_cast<size_t>(member) * a.E + e0 + tid) * a.trace_T + t) * 4;
                    tr[0] = cps.x; tr[1] = cps.xd; tr[2] = cps.th; tr[3] = cps.thd;
                }
            }
            __syncthreads();
        } else {
            if (tid < nE) {                                    // reward on (x_t, a_t)
                float xx = 0.f, aa = 0.f;
                for (uint32_t k = 0; k < kTlNx; ++k) xx = fmaf(obs[k * EB + tid], obs[k * EB + tid], xx);
                for (uint32_t k = 0; k < kTlNa; ++k) aa = fmaf(act[k * EB + tid], act[k * EB + tid], aa);
                ret += -xx - 0.01f * aa;
            }
            const float* A = tcon;
            const float* B = tcon + kTlNx * kTlNx;
            for (uint32_t item = tid; item < kTlNx * nE; item += blockDim.x) {
                const uint32_t i = item / nE, e = item % nE;
                float acc = 0.f;
                for (uint32_t k = 0; k < kTlNx; ++k) acc = fmaf(A[i * kTlNx + k], obs[k * EB + e], acc);
                for (uint32_t k = 0; k < kTlNa; ++k) acc = fmaf(B[i * kTlNa + k], act[k * EB + e], acc);
                nxt[i * EB + e] = tanhf(acc);
            }
            __syncthreads();
            for (uint32_t item = tid; item < kTlNx * nE; item += blockDim.x) {
                const uint32_t i = item / nE, e = item % nE;
                const float xv = nxt[i * EB + e];
                obs[i * EB + e] = xv;
                if (a.trace && t < a.trace_T)
                    a.trace[((static_cast<size_t>(member) * a.E + e0 + e) * a.trace_T + t) * kTlNx + i] = xv;
            }
            __syncthreads();
        }
    }

    if (tid < nE) rets[tid] = ret;
    __syncthreads();
    if (tid == 0) {
        float s = 0.f;
        for (uint32_t e = 0; e < nE; ++e) s += rets[e];
        if (EVO_IN_BOUNDS(status, EVO_SITE_FIT_PARTIAL, static_cast<size_t>(member) * a.n_eb + eb, static_cast<size_t>(a.P) * a.n_eb))
            a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = s;
    }
}

// fitness[m] = (sum of the member's episode-block partial sums, in block order) / E
__global__ void k_fitness_finalize(const float* __restrict__ partial, uint32_t P, uint32_t n_eb,
                                   uint32_t E, float* __restrict__ fitness)
{
    dep_wait();
    dep_trigger();                       // the ranking that follows may be set up
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= P) return;
    float s = 0.f;
    for (uint32_t b = 0; b < n_eb; ++b) s += partial[static_cast<size_t>(m) * n_eb + b];
    fitness[m] = s / static_cast<float>(E);
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static uint32_t param_count(const evo_config& cfg)
{
    uint32_t n = 0;
    for (uint32_t l = 0; l < cfg.n_layers; ++l)
        n += cfg.layer_sizes[l + 1] * cfg.layer_sizes[l] + cfg.layer_sizes[l + 1];
    return n;
}

bool rollout_mlp_supported(const evo_config& cfg)
{
    if (cfg.policy_kind != EVO_POLICY_MLP) return false;
    if (cfg.n_layers < 1 || cfg.n_layers > EVO_MAX_LAYERS) return false;
    for (uint32_t l = 0; l <= cfg.n_layers; ++l)
        if (cfg.layer_sizes[l] < 1 || cfg.layer_sizes[l] > 1024) return false;
    if (param_count(cfg) != cfg.param_dim) return false;
    if (cfg.task_kind == EVO_TASK_CARTPOLE)
        return cfg.layer_sizes[0] == 5 && cfg.layer_sizes[cfg.n_layers] == 1;
    if (cfg.task_kind == EVO_TASK_TANH_LINEAR)
        return cfg.layer_sizes[0] == kTlNx && cfg.layer_sizes[cfg.n_layers] == kTlNa;
    return false;
}

int rollout_mlp_tiled_shape(uint32_t task, uint32_t n_layers, const uint32_t* sizes);
uint32_t rollout_mlp_tiled_eb(int shape, uint32_t episodes);
int launch_rollout_mlp_tiled(cudaStream_t st, const RolloutMlpArgs& a, DeviceStatus* status);
bool rollout_tl_tc_supported(const RolloutMlpArgs& a);
int launch_rollout_tl_tc(cudaStream_t st, const RolloutMlpArgs& a, DeviceStatus* status);

static bool use_tiled(uint32_t task, uint32_t n_layers, const uint32_t* sizes, uint32_t choice)
{
    return choice != EVO_ROLLOUT_GENERIC && rollout_mlp_tiled_shape(task, n_layers, sizes) >= 0;
}

void rollout_mlp_plan(const evo_config& cfg, uint32_t* EB, uint32_t* n_eb)
{
    if (use_tiled(cfg.task_kind, cfg.n_layers, cfg.layer_sizes, cfg.rollout_kernel)) {
        *EB = rollout_mlp_tiled_eb(rollout_mlp_tiled_shape(cfg.task_kind, cfg.n_layers, cfg.layer_sizes), cfg.episodes);
        *n_eb = (cfg.episodes + *EB - 1u) / *EB;
        return;
    }
    uint32_t eb = cfg.episodes < 32u ? cfg.episodes : 32u;
    // few members: split the episodes of a member over more blocks to fill the SMs
    while (eb > 4u && static_cast<uint64_t>(cfg.pop_size) * ((cfg.episodes + eb - 1u) / eb) < 4u * 148u)
        eb = (eb + 1u) / 2u;
    *EB = eb;
    *n_eb = (cfg.episodes + eb - 1u) / eb;
}

static size_t generic_smem_bytes(const RolloutMlpArgs& a, bool with_weights)
{
    uint32_t n_params = 0;
    for (uint32_t l = 0; l < a.n_layers; ++l) n_params += a.sizes[l + 1] * a.sizes[l] + a.sizes[l + 1];
    size_t f = 2u * a.max_width * a.EB + a.sizes[0] * a.EB + a.sizes[a.n_layers] * a.EB + a.EB;
    if (a.task == EVO_TASK_TANH_LINEAR) f += kTlNx * a.EB + kTlNx * (kTlNx + kTlNa);
    if (with_weights) f += n_params;
    return f * sizeof(float);
}

int launch_rollout_mlp(cudaStream_t st, const RolloutMlpArgs& a_in, uint32_t kernel_choice, float* fitness,
                       DeviceStatus* status)
{
    RolloutMlpArgs a = a_in;
    int launches = 0;
    const bool tiled_ok = rollout_mlp_tiled_shape(a.task, a.n_layers, a.sizes) >= 0;
    if (kernel_choice == EVO_ROLLOUT_TILED && !tiled_ok) return -2;
    if (kernel_choice == EVO_ROLLOUT_AUTO && rollout_tl_tc_supported(a)) {
        // the large tanh-linear policy: wide layers on the tensor cores (TILED keeps the fp32-pipe kernel)
        const int r = launch_rollout_tl_tc(st, a, status);
        if (r < 0) return r;
        launches += r;
    } else if (tiled_ok && kernel_choice != EVO_ROLLOUT_GENERIC) {
        const int r = launch_rollout_mlp_tiled(st, a, status);
        if (r < 0) return r;
        launches += r;
    } else {
        size_t bytes = generic_smem_bytes(a, true);
        a.weights_in_smem = 1;
        if (bytes > 200u * 1024u) { a.weights_in_smem = 0; bytes = generic_smem_bytes(a, false); }
        if (bytes > 200u * 1024u) return -2;
        if (!a.attr_done &&
            cudaFuncSetAttribute(k_rollout_mlp_generic, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(bytes)) != cudaSuccess) return -1;
        dim3 grid(a.P, a.n_eb);
        k_rollout_mlp_generic<<<grid, kGenericThreads, bytes, st>>>(a, status);
        if (cudaGetLastError() != cudaSuccess) return -1;
        launches += 1;
    }
    if (launch_dependent(k_fitness_finalize, dim3((a.P + 255u) / 256u), dim3(256), 0, st, a.fit_partial, a.P, a.n_eb, a.E,
                         fitness) != cudaSuccess) return -1;
    return launches + 1;
}

}  // namespace evo
