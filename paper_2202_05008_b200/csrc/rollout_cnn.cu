// Supervised single-step "rollout": every member's convolutional policy is run on the bound
// batch and scored by -mean cross-entropy (paper Section 3: supervised learning tasks are
// single-step tasks; MNIST-shaped ConvNet example).  Network: conv 1->8 5x5 valid + ReLU +
// 2x2 max-pool, conv 8->16 5x5 valid + ReLU + 2x2 max-pool, linear 256->10.  Operands of the
// three contractions are rounded to bf16 (round to nearest even), accumulation is fp32.
#include "internal.h"
#include <cuda_bf16.h>

namespace evo {

constexpr int kCnnThreads = 256;
constexpr int kCnnImgsPerBlock = 8;

__device__ __forceinline__ float bf16r(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// CUDA-core version: block = (member, tile of images); the member's weights stay in shared
// memory for the whole tile.
__global__ void __launch_bounds__(kCnnThreads)
k_cnn_simple(const float* __restrict__ theta, uint32_t ldD, const float* __restrict__ images,
             const int32_t* __restrict__ labels, uint32_t batch, uint32_t n_tiles,
             float* __restrict__ partial)
{
    __shared__ float w1[200], b1[8], w2[3200], b2[16], wf[2560], bfc[10];
    __shared__ float img[784], p1[1152], p2[256], logits[10];
    __shared__ float loss_sum;
    const uint32_t member = blockIdx.x, tile = blockIdx.y, tid = threadIdx.x;
    const float* p = theta + static_cast<size_t>(member) * ldD;
    for (uint32_t i = tid; i < 200; i += kCnnThreads) w1[i] = bf16r(p[i]);
    if (tid < 8) b1[tid] = p[200 + tid];
    for (uint32_t i = tid; i < 3200; i += kCnnThreads) w2[i] = bf16r(p[208 + i]);
    if (tid < 16) b2[tid] = p[3408 + tid];
    for (uint32_t i = tid; i < 2560; i += kCnnThreads) wf[i] = bf16r(p[3424 + i]);
    if (tid < 10) bfc[tid] = p[5984 + tid];
    if (tid == 0) loss_sum = 0.f;

    const uint32_t i0 = tile * kCnnImgsPerBlock;
    const uint32_t i1 = min(batch, i0 + kCnnImgsPerBlock);
    for (uint32_t im = i0; im < i1; ++im) {
        __syncthreads();
        const float* src = images + static_cast<size_t>(im) * 784;
        for (uint32_t i = tid; i < 784; i += kCnnThreads) img[i] = bf16r(src[i]);
        __syncthreads();
        // conv1 + pool: one pooled output (channel, py, px) per item
        for (uint32_t o = tid; o < 1152; o += kCnnThreads) {
            const uint32_t c = o / 144, py = (o % 144) / 12, px = o % 12;
            const float* wc = w1 + c * 25;
            float best = -3.0e38f;
#pragma unroll
            for (int dy = 0; dy < 2; ++dy)
#pragma unroll
                for (int dx = 0; dx < 2; ++dx) {
                    const float* ip = img + (2 * py + dy) * 28 + (2 * px + dx);
                    float acc = 0.f;
#pragma unroll
                    for (int kh = 0; kh < 5; ++kh)
#pragma unroll
                        for (int kw = 0; kw < 5; ++kw) acc = fmaf(wc[kh * 5 + kw], ip[kh * 28 + kw], acc);
                    best = fmaxf(best, acc);
                }
            p1[o] = bf16r(fmaxf(best + b1[c], 0.f));
        }
        __syncthreads();
        // conv2 + pool: 256 pooled outputs, flattened (channel, y, x)
        {
            const uint32_t o = tid;
            const uint32_t c = o / 16, py = (o % 16) / 4, px = o % 4;
            float acc[4] = { 0.f, 0.f, 0.f, 0.f };
            for (int ic = 0; ic < 8; ++ic) {
                const float* wc = w2 + (c * 8 + ic) * 25;
                const float* ip = p1 + ic * 144 + (2 * py) * 12 + 2 * px;
#pragma unroll
                for (int kh = 0; kh < 5; ++kh)
#pragma unroll
                    for (int kw = 0; kw < 5; ++kw) {
                        const float wv = wc[kh * 5 + kw];
                        acc[0] = fmaf(wv, ip[(kh) * 12 + kw], acc[0]);
                        acc[1] = fmaf(wv, ip[(kh) * 12 + kw + 1], acc[1]);
                        acc[2] = fmaf(wv, ip[(kh + 1) * 12 + kw], acc[2]);
                        acc[3] = fmaf(wv, ip[(kh + 1) * 12 + kw + 1], acc[3]);
                    }
            }
            const float best = fmaxf(fmaxf(acc[0], acc[1]), fmaxf(acc[2], acc[3]));
            p2[o] = bf16r(fmaxf(best + b2[c], 0.f));
        }
        __syncthreads();
        // linear 256 -> 10: one warp per class
        for (uint32_t cls = tid / 32; cls < 10; cls += kCnnThreads / 32) {
            const uint32_t lane = tid % 32;
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = fmaf(wf[cls * 256 + lane + 32 * k], p2[lane + 32 * k], acc);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) logits[cls] = acc + bfc[cls];
        }
        __syncthreads();
        if (tid == 0) {
            float mx = logits[0];
            for (int k = 1; k < 10; ++k) mx = fmaxf(mx, logits[k]);
            float se = 0.f;
            for (int k = 0; k < 10; ++k) se += expf(logits[k] - mx);
            loss_sum += (mx + logf(se)) - logits[labels[im]];
        }
    }
    __syncthreads();
    if (tid == 0) partial[static_cast<size_t>(member) * n_tiles + tile] = loss_sum;
}

__global__ void k_cnn_finalize(const float* __restrict__ partial, uint32_t P, uint32_t n_tiles,
                               uint32_t batch, float* __restrict__ fitness)
{
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= P) return;
    float s = 0.f;
    for (uint32_t t = 0; t < n_tiles; ++t) s += partial[static_cast<size_t>(m) * n_tiles + t];
    fitness[m] = -s / static_cast<float>(batch);
}

size_t cnn_scratch_bytes(uint32_t P, uint32_t batch)
{
    const size_t n_tiles = (batch + kCnnImgsPerBlock - 1) / kCnnImgsPerBlock;
    return static_cast<size_t>(P) * n_tiles * sizeof(float);
}

int launch_rollout_cnn(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P,
                       const float* images, const int32_t* labels, uint32_t batch, void* scratch,
                       float* fitness)
{
    const uint32_t n_tiles = (batch + kCnnImgsPerBlock - 1) / kCnnImgsPerBlock;
    float* partial = static_cast<float*>(scratch);
    dim3 grid(P, n_tiles);
    k_cnn_simple<<<grid, kCnnThreads, 0, st>>>(theta, ldD, images, labels, batch, n_tiles, partial);
    if (cudaGetLastError() != cudaSuccess) return -1;
    k_cnn_finalize<<<(P + 255u) / 256u, 256, 0, st>>>(partial, P, n_tiles, batch, fitness);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 2;
}

}  // namespace evo
