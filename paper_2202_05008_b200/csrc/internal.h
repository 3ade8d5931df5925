// Internal declarations shared by the host API (evo.cu) and the kernel files.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/evo.h"

namespace evo {

// Device-resident control block at the start of the workspace.
struct DeviceStatus {
    uint32_t sticky;        // OR of (1u << evo_status) for conditions raised on the device
    uint32_t nonfinite;     // set by the rank kernel of the current tell, cleared by its finish
    uint32_t adam_step;     // t
    uint32_t generation;    // counter word of every random stream; advanced by the kernel that closes a tell
    uint32_t wait_cycles_log2;  // every bounded device-side wait gives up after 2^this SM clocks
    uint32_t debug_flags;   // EVO_DEBUG_* bits of the configuration
    uint32_t bounds_site;   // checked build: first store site whose index left its array (0 = none)
    uint32_t bounds_index_lo, bounds_index_hi;   // ... and that index
    uint32_t reserved;
};

// Checked build (-DEVO_DEBUG, libevo_debug.so): a global store whose index lies outside its array is
// not executed; the first such site and index are recorded in the status block and the sticky
// EVO_ERR_CUDA bit is raised.  In the normal build the macro is the constant true.
enum { EVO_SITE_ASK_THETA = 1, EVO_SITE_ASK_EPS = 2, EVO_SITE_RANK = 3, EVO_SITE_GRAD_PARTIAL = 4,
       EVO_SITE_UPDATE = 5, EVO_SITE_FIT_PARTIAL = 6, EVO_SITE_TRACE = 7, EVO_SITE_FITNESS = 8 };
#ifdef EVO_DEBUG
__device__ __forceinline__ bool debug_in_bounds(const DeviceStatus* st, uint32_t site, unsigned long long idx,
                                                unsigned long long limit)
{
    if (idx < limit) return true;
    DeviceStatus* s = const_cast<DeviceStatus*>(st);
    if (atomicCAS(&s->bounds_site, 0u, site) == 0u) {
        s->bounds_index_lo = static_cast<uint32_t>(idx);
        s->bounds_index_hi = static_cast<uint32_t>(idx >> 32);
    }
    atomicOr(&s->sticky, 1u << EVO_ERR_CUDA);
    return false;
}
#define EVO_IN_BOUNDS(st, site, idx, limit) ::evo::debug_in_bounds(st, site, idx, limit)
constexpr size_t kCanaryBytes = 256;      // guard words behind every workspace region
#else
#define EVO_IN_BOUNDS(st, site, idx, limit) true
constexpr size_t kCanaryBytes = 0;
#endif
constexpr int kMaxRegions = 24;

constexpr uint32_t kTlNx = 28;   // tanh-linear task: state width
constexpr uint32_t kTlNa = 8;    // tanh-linear task: action width
constexpr uint32_t kCnnParams = 5994;
constexpr uint32_t kMaxParamDim = 1u << 30;   // keeps ldD = round_up(D, 32) and 4 * ldD inside 32 bits

struct RolloutMlpArgs {
    const float* theta;          // [P][ldD]
    float*       fit_partial;    // [P][n_episode_blocks] sums of episode returns
    float*       trace;          // nullable
    const float* task_const;     // tanh-linear: A[28][28] then B[28][8]
    uint32_t P, ldD;
    uint32_t n_layers;
    uint32_t sizes[EVO_MAX_LAYERS + 1];
    uint32_t max_width;
    float    action_scale;
    uint32_t task;
    uint32_t E, T, EB, n_eb;     // episodes, horizon, episodes per block, blocks per member
    uint32_t trace_T;
    uint32_t k0, k1;             // the generation is read from the device status by the kernels
    float    tp[16];
    uint32_t weights_in_smem;
    uint32_t attr_done;          // the kernel's dynamic shared-memory limit was raised by an earlier launch of this solver
};

struct Layout {                  // byte offsets into the workspace
    size_t status, center, m, v, g, sigma, theta, eps, u, rank, grad_partial, sigma_partial, grad_sum,
           sigma_sum, norms,
           fit_partial, task_const, cnn_scratch, total;
    uint32_t ldD, grad_splits, n_eb, EB;
    size_t canary[kMaxRegions];  // checked build: offset of the guard words behind each region, in layout order
    int    n_canaries;
};

// ---- launchers (each returns the number of kernels it launched, or -1 on a launch error) ----
int launch_init(cudaStream_t st, float* center, float* m, float* v, float* g, float* sigma_vec,
                float sigma, uint32_t D, uint32_t ldD, DeviceStatus* status, uint32_t wait_cycles_log2,
                uint32_t debug_flags);
int launch_task_constants(cudaStream_t st, uint32_t task, uint32_t k0, uint32_t k1, float* task_const);
int launch_ask(cudaStream_t st, const float* center, const float* sigma_vec, uint32_t k0, uint32_t k1,
               const DeviceStatus* status, uint32_t pair0, uint32_t H, uint32_t D, uint32_t ldD, float* theta,
               float* eps);
int launch_rank(cudaStream_t st, const float* fitness, uint32_t P, int32_t* rank, float* u,
                DeviceStatus* status);
struct TellArgs {
    const float* u;               // centred-rank weights [P]
    const float* eps;             // stored noise, or NULL = regenerate from the counters
    uint32_t k0, k1, H, D, ldD, splits;   // H = pairs summed here (the shard's)
    uint32_t pair0, P;            // first global pair of the shard; global population size
    double* partial;              // [splits][ldD] fp64 partial sums of the centre gradient
    float*  sigma_partial;        // [splits][ldD] fp32 partial sums of the sigma gradient, or NULL
    double* norms;                // scratch for ClipUp's two vector norms
    float*  sigma_vec;            // [ldD]
    float   lr, beta1, beta2, adam_eps;
    uint32_t optimizer;
    float   clipup_momentum, clipup_max_speed;
    float   sigma_lr, sigma_max_change;
    float*  center; float* m; float* v; float* g;
    DeviceStatus* status;
};
int launch_gradient_update(cudaStream_t st, const TellArgs& a);
// the two halves of the sharded tell: partial sums -> reduce buffers; reduce buffers -> update
int launch_gradient_sums(cudaStream_t st, const TellArgs& a, double* grad_sum, float* sigma_sum);
int launch_update_from_sums(cudaStream_t st, const TellArgs& a, const double* grad_sum, const float* sigma_sum);
size_t clipup_norm_doubles(uint32_t ldD);
uint32_t gradient_splits(uint32_t H, uint32_t ldD);

int  launch_rollout_mlp(cudaStream_t st, const RolloutMlpArgs& a, uint32_t kernel_choice,
                        float* fitness, DeviceStatus* status);
bool rollout_mlp_supported(const evo_config& cfg);
void rollout_mlp_plan(const evo_config& cfg, uint32_t* EB, uint32_t* n_eb);

size_t cnn_scratch_bytes(uint32_t P, uint32_t batch);
size_t cnn_tc_scratch_bytes(uint32_t P, uint32_t batch);
int launch_rollout_cnn_tc(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, const float* images,
                          const int32_t* labels, uint32_t batch, void* scratch, float* fitness,
                          DeviceStatus* status);
int launch_rollout_cnn(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P,
                       const float* images, const int32_t* labels, uint32_t batch, void* scratch,
                       float* fitness);

uint32_t s2s_param_count(uint32_t h);
bool s2s_supported(uint32_t h, uint32_t nd, uint32_t B);
size_t s2s_scratch_bytes(uint32_t P, uint32_t B);
// logits (nullable): [P][B][nd+1][12], written by the CUDA-core kernel only
int launch_rollout_s2s(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, uint32_t h, uint32_t nd,
                       uint32_t B, uint32_t k0, uint32_t k1, uint32_t kernel_choice,
                       void* scratch, float* fitness, float* logits, DeviceStatus* status);

bool paint_supported(uint32_t param_dim, uint32_t W, uint32_t H);
size_t paint_scratch_bytes(uint32_t P, uint32_t W, uint32_t H);
// canvas (nullable): [P][H][W][3]
int launch_rollout_paint(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, uint32_t param_dim,
                         uint32_t W, uint32_t H, float background, const float* target, void* scratch,
                         float* fitness, float* canvas);

// ------------------------------------------------------------------------------------------
// Programmatic dependent launch.  The small kernels of a generation follow one another in one
// stream, and between two of them the launch of the second costs about as much as the kernel itself
// runs.  A kernel launched with launch_dependent may be set up while its predecessor is still
// running; it MUST call dep_wait() before it reads or writes anything (every thread, before any
// return): that waits for the predecessor to have completed, and so, one after the other, for
// everything before it.  A kernel lets its successor be set up with dep_trigger().  After a kernel that
// never triggers, or after a copy, the launch is an ordinary one.
// ------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

}  // namespace evo
