// Register-only fp32 FMA chains: the measured counterpart of the nominal fp32 peak
// (SMs x 128 lanes x 2 flop x clock) that the roll-out kernels are reported against.
// Every thread runs kChains independent fused multiply-adds per iteration on values that
// never leave registers; one store at the end keeps the work observable.
#include "internal.h"

namespace evo {

constexpr int kChains = 16;

__global__ void __launch_bounds__(1024)
k_fma_probe(float* __restrict__ sink, uint32_t iters, float a, float b)
{
    float x[kChains];
#pragma unroll
    for (int i = 0; i < kChains; ++i) x[i] = static_cast<float>(threadIdx.x + i) * 1e-3f;
    for (uint32_t it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kChains; ++i) x[i] = fmaf(x[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kChains; ++i) s += x[i];
    sink[static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x] = s;
}

}  // namespace evo

extern "C" evo_status evo_fma_probe(float* d_sink, uint32_t blocks, uint32_t threads, uint32_t iters,
                                    void* cuda_stream, uint64_t* flops)
{
    if (!d_sink || !flops || blocks == 0 || threads == 0 || threads > 1024 || (threads & 31u) || iters == 0)
        return EVO_ERR_INVALID_ARG;
    // a contraction (|a| < 1) keeps every chain finite for any iteration count
    evo::k_fma_probe<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(d_sink, iters, 0.999f, 1e-3f);
    if (cudaGetLastError() != cudaSuccess) return EVO_ERR_CUDA;
    *flops = 2ull * evo::kChains * iters * static_cast<uint64_t>(blocks) * threads;
    return EVO_OK;
}
