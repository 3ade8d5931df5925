// evo_es_gradient_static: the ES gradient for callers that may not allocate device memory.
//
// Some users of this library run where nobody is allowed to call cudaMalloc once the program
// is up: a long-running service that hands out all device memory at start-up so that it can
// never hit an out-of-memory error or fragment later, or a plug-in living inside another
// framework whose allocator owns the whole GPU.  Such a caller cannot provide the workspace
// blob that evo_create asks for, so this one entry point carries its own scratch: the split
// partial sums of the gradient reduction live in a fixed array that is part of the loaded
// library image (every GPU that loads the library holds it until the process exits).
#include "internal.h"

#include <mutex>

namespace evo {

// 4 MiB of fp64 partial sums: splits * ldD <= 524,288 values.
constexpr size_t kStaticScratchDoubles = EVO_STATIC_SCRATCH_BYTES / sizeof(double);
static __device__ __align__(256) double g_static_scratch[kStaticScratchDoubles];

// In host code the name above is only a handle for the runtime, not a device address; the
// address each device maps it to is looked up once per device and cached here.  The cached
// address belongs to the device's primary context: after cudaDeviceReset it is stale, so a
// process that resets a device must not call this entry point on it again.
constexpr int kMaxDevices = 64;
static double*    g_scratch_ptr[kMaxDevices] = {};
static std::mutex g_scratch_mutex;

static double* static_scratch_for_current_device(cudaError_t* err)
{
    int dev = -1;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= kMaxDevices) { *err = cudaErrorInvalidDevice; return nullptr; }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        double* p = nullptr;
        *err = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (*err != cudaSuccess) return nullptr;
        g_scratch_ptr[dev] = p;
    }
    return g_scratch_ptr[dev];
}

// partial[s][d] = sum over the pairs of split s of (u[2j] - u[2j+1]) * eps[j][d]   (fp64)
__global__ void __launch_bounds__(128)
k_grad_partial_static(const float* __restrict__ u, const float* __restrict__ eps, uint32_t H,
                      uint32_t D, size_t ld_eps, uint32_t ldS, uint32_t pairs_per_split,
                      double* __restrict__ partial)
{
    const uint32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= ldS) return;
    const uint32_t j0 = blockIdx.y * pairs_per_split;
    const uint32_t j1 = min(H, j0 + pairs_per_split);
    double acc0 = 0.0, acc1 = 0.0;
    if (d < D) {
        uint32_t j = j0;
        for (; j + 2u <= j1; j += 2u) {
            const double w0 = static_cast<double>(u[2u * j]) - static_cast<double>(u[2u * j + 1u]);
            const double w1 = static_cast<double>(u[2u * j + 2u]) - static_cast<double>(u[2u * j + 3u]);
            acc0 = fma(w0, static_cast<double>(__ldcs(eps + static_cast<size_t>(j) * ld_eps + d)), acc0);
            acc1 = fma(w1, static_cast<double>(__ldcs(eps + static_cast<size_t>(j + 1u) * ld_eps + d)), acc1);
        }
        if (j < j1) {
            const double w0 = static_cast<double>(u[2u * j]) - static_cast<double>(u[2u * j + 1u]);
            acc0 = fma(w0, static_cast<double>(__ldcs(eps + static_cast<size_t>(j) * ld_eps + d)), acc0);
        }
    }
    // every word the second kernel reads is written here, so stale contents never leak in
    partial[static_cast<size_t>(blockIdx.y) * ldS + d] = acc0 + acc1;
}

__global__ void __launch_bounds__(256)
k_grad_sum_static(const double* __restrict__ partial, uint32_t splits, uint32_t D, uint32_t ldS,
                  double scale, float* __restrict__ g)
{
    const uint32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= D) return;
    double s = 0.0;
    for (uint32_t k = 0; k < splits; ++k) s += partial[static_cast<size_t>(k) * ldS + d];
    g[d] = static_cast<float>(s * scale);
}

}  // namespace evo

using namespace evo;

extern "C" evo_status evo_es_gradient_static(const float* d_u, const float* d_eps, uint32_t pop_size,
                                             uint32_t param_dim, size_t ld_eps, float sigma,
                                             float* d_gradient, void* cuda_stream)
{
    if (!d_u || !d_eps || !d_gradient) return EVO_ERR_INVALID_ARG;
    if (pop_size < 2 || (pop_size & 1u) || param_dim < 1 || ld_eps < param_dim) return EVO_ERR_INVALID_ARG;
    const uint32_t H = pop_size / 2u;
    // the size check comes first and in 64 bits: rounding a huge param_dim up must not wrap to 0
    if ((static_cast<size_t>(param_dim) + 31u) / 32u * 32u > kStaticScratchDoubles) return EVO_ERR_WORKSPACE;
    const uint32_t ldS = (param_dim + 31u) / 32u * 32u;             // row pitch inside the scratch
    // as many splits as the plan for this shape wants, but no more than the fixed array holds
    uint32_t splits = gradient_splits(H, ldS);
    const size_t fit = kStaticScratchDoubles / ldS;
    if (splits > fit) splits = static_cast<uint32_t>(fit);
    const uint32_t pps = (H + splits - 1u) / splits;
    const uint32_t used = (H + pps - 1u) / pps;

    cudaError_t err;
    double* scratch = static_scratch_for_current_device(&err);
    if (!scratch) return EVO_ERR_CUDA;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    dim3 grid((ldS + 127u) / 128u, used);
    k_grad_partial_static<<<grid, 128, 0, st>>>(d_u, d_eps, H, param_dim, ld_eps, ldS, pps, scratch);
    if (cudaGetLastError() != cudaSuccess) return EVO_ERR_CUDA;
    const double scale = static_cast<double>(sigma) / static_cast<double>(pop_size);
    k_grad_sum_static<<<(param_dim + 255u) / 256u, 256, 0, st>>>(scratch, used, param_dim, ldS, scale,
                                                                 d_gradient);
    if (cudaGetLastError() != cudaSuccess) return EVO_ERR_CUDA;
    return EVO_OK;
}
