// Measurement aid of bench.py, not part of the library: register-only fp32 FMA chains, the
// measured counterpart of the nominal fp32 peak (SMs x 128 lanes x 2 flop x clock) that the
// roll-out kernels are reported against.  Every thread runs kChains independent fused
// multiply-adds per iteration on values that never leave registers; one store at the end keeps
// the work observable.  Built into libbench_fma_probe.so beside bench.py.
#include <cstdint>
#include <cuda_runtime.h>

namespace {

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

}  // namespace

// Launches blocks x threads threads on cuda_stream (asynchronous); d_sink[blocks*threads] is
// caller-owned device memory; *flops receives the floating-point operations of the launch
// (2 per FMA).  Returns 0, 1 for a bad argument (NULL pointer, zero size, threads not a multiple
// of 32 or above 1024), 4 when the launch failed.
extern "C" int bench_fma_probe(float* d_sink, uint32_t blocks, uint32_t threads, uint32_t iters,
                               void* cuda_stream, uint64_t* flops)
{
    if (!d_sink || !flops || blocks == 0 || threads == 0 || threads > 1024 || (threads & 31u) || iters == 0)
        return 1;
    // a contraction (|a| < 1) keeps every chain finite for any iteration count
    k_fma_probe<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(d_sink, iters, 0.999f, 1e-3f);
    if (cudaGetLastError() != cudaSuccess) return 4;
    *flops = 2ull * kChains * iters * static_cast<uint64_t>(blocks) * threads;
    return 0;
}
