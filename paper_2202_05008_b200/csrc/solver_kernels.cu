// Solver kernels: ask (antithetic sampling), centred rank, ES gradient (stored or regenerated
// noise) and the Adam ascent step.  Paper Section 4 (NEAlgorithm ask / tell), Section 2
// ("Modern ML Optimizers"); the algorithm is PGPE with symmetric sampling (Section 5).
#include "internal.h"
#include "noise.cuh"

namespace evo {

// ------------------------------------------------------------------------------------------
// init / task constants
// ------------------------------------------------------------------------------------------
__global__ void k_init(float* center, float* m, float* v, float* g, float* sigma_vec, float sigma,
                       uint32_t D, uint32_t ldD, DeviceStatus* status, uint32_t wait_cycles_log2,
                       uint32_t debug_flags)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < ldD) { center[i] = 0.f; m[i] = 0.f; v[i] = 0.f; g[i] = 0.f; sigma_vec[i] = (i < D) ? sigma : 0.f; }
    if (i == 0) {
        status->sticky = 0; status->nonfinite = 0; status->adam_step = 0; status->generation = 0;
        status->wait_cycles_log2 = wait_cycles_log2; status->debug_flags = debug_flags;
        status->bounds_site = 0; status->bounds_index_lo = 0; status->bounds_index_hi = 0; status->reserved = 0;
    }
}

int launch_init(cudaStream_t st, float* center, float* m, float* v, float* g, float* sigma_vec,
                float sigma, uint32_t D, uint32_t ldD, DeviceStatus* status, uint32_t wait_cycles_log2,
                uint32_t debug_flags)
{
    k_init<<<(ldD + 255) / 256, 256, 0, st>>>(center, m, v, g, sigma_vec, sigma, D, ldD, status,
                                              wait_cycles_log2, debug_flags);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// Tanh-linear task constants: A[28][28] = z * fp32(0.9/sqrt(28)), B[28][8] = z * fp32(1/sqrt(8)),
// z from stream 4 (row 0 = A, row 1 = B), generation 0.
__global__ void k_tanh_linear_constants(PhiloxKey key, float* out)
{
    const uint32_t quad = threadIdx.x;
    constexpr uint32_t qa = kTlNx * kTlNx / 4, qb = kTlNx * kTlNa / 4;
    if (quad < qa) {
        const float4 z = stream_normal4(key, 4u, 0u, 0u, quad);
        const float sc = __uint_as_float(0x3E2E2A81u);
        float4 r = make_float4(__fmul_rn(z.x, sc), __fmul_rn(z.y, sc), __fmul_rn(z.z, sc), __fmul_rn(z.w, sc));
        reinterpret_cast<float4*>(out)[quad] = r;
    } else if (quad < qa + qb) {
        const float4 z = stream_normal4(key, 4u, 0u, 1u, quad - qa);
        const float sc = __uint_as_float(0x3EB504F3u);
        float4 r = make_float4(__fmul_rn(z.x, sc), __fmul_rn(z.y, sc), __fmul_rn(z.z, sc), __fmul_rn(z.w, sc));
        reinterpret_cast<float4*>(out)[quad] = r;
    }
}

int launch_task_constants(cudaStream_t st, uint32_t task, uint32_t k0, uint32_t k1, float* task_const)
{
    if (task != EVO_TASK_TANH_LINEAR) return 0;
    k_tanh_linear_constants<<<1, 256, 0, st>>>(philox_key(k0, k1), task_const);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// ------------------------------------------------------------------------------------------
// ask: one thread per (column quad, chunk of pairs).  Writes are 128-bit and coalesced along
// the row; the centre quad is loaded once per thread and reused for all pairs of the chunk.
// ------------------------------------------------------------------------------------------
constexpr uint32_t kAskPairsPerThread = 8;

__global__ void __launch_bounds__(256, 8)
k_ask(const float* __restrict__ center, const float* __restrict__ sigma_vec, PhiloxKey key,
      const DeviceStatus* __restrict__ status, uint32_t pair0, uint32_t H, uint32_t D, uint32_t ldD, float* __restrict__ theta, float* __restrict__ eps)
{
    dep_wait();
    dep_trigger();                       // the roll-out that follows may be set up
    const uint32_t quad = blockIdx.x * blockDim.x + threadIdx.x;
    if (quad * 4u >= ldD) return;
    const uint32_t generation = status->generation;
    const uint32_t d0 = quad * 4u;
    const float4 c = reinterpret_cast<const float4*>(center)[quad];
    const float4 sg = reinterpret_cast<const float4*>(sigma_vec)[quad];      // one sigma per dimension
    const bool full = d0 + 4u <= D;
    for (uint32_t j = blockIdx.y * kAskPairsPerThread; j < H; j += gridDim.y * kAskPairsPerThread) {
        const uint32_t jend = min(j + kAskPairsPerThread, H);
        for (uint32_t jj = j; jj < jend; ++jj) {
            float4 z = stream_normal4(key, 0u, generation, pair0 + jj, quad);   // counters use the global pair
            if (!full) {                       // ragged tail and padding columns carry zeros
                if (d0 + 0u >= D) z.x = 0.f;
                if (d0 + 1u >= D) z.y = 0.f;
                if (d0 + 2u >= D) z.z = 0.f;
                if (d0 + 3u >= D) z.w = 0.f;
            }
            const float4 tp = make_float4(__fmaf_rn(sg.x, z.x, c.x), __fmaf_rn(sg.y, z.y, c.y),
                                          __fmaf_rn(sg.z, z.z, c.z), __fmaf_rn(sg.w, z.w, c.w));
            const float4 tm = make_float4(__fmaf_rn(-sg.x, z.x, c.x), __fmaf_rn(-sg.y, z.y, c.y),
                                          __fmaf_rn(-sg.z, z.z, c.z), __fmaf_rn(-sg.w, z.w, c.w));
            float* row = theta + static_cast<size_t>(2u * jj) * ldD + d0;
            if (EVO_IN_BOUNDS(status, EVO_SITE_ASK_THETA, static_cast<size_t>(2u * jj + 1u) * ldD + d0 + 3u,
                              static_cast<size_t>(2u * H) * ldD)) {
                __stcs(reinterpret_cast<float4*>(row), tp);
                __stcs(reinterpret_cast<float4*>(row + ldD), tm);
            }
            if (eps && EVO_IN_BOUNDS(status, EVO_SITE_ASK_EPS, static_cast<size_t>(jj) * ldD + d0 + 3u,
                                     static_cast<size_t>(H) * ldD))
                __stcs(reinterpret_cast<float4*>(eps + static_cast<size_t>(jj) * ldD + d0), z);
        }
    }
}

int launch_ask(cudaStream_t st, const float* center, const float* sigma_vec, uint32_t k0, uint32_t k1,
               const DeviceStatus* status, uint32_t pair0, uint32_t H, uint32_t D, uint32_t ldD, float* theta,
               float* eps)
{
    const uint32_t quads = ldD / 4u;
    dim3 grid((quads + 255u) / 256u, (H + kAskPairsPerThread - 1u) / kAskPairsPerThread);
    if (grid.y > 65535u) grid.y = 65535u;
    return launch_dependent(k_ask, grid, dim3(256), 0, st, center, sigma_vec, philox_key(k0, k1), status, pair0, H, D, ldD,
                            theta, eps) == cudaSuccess ? 1 : -1;
}

// ------------------------------------------------------------------------------------------
// centred rank by counting: rank_m = #{k : f_k < f_m or (f_k == f_m and k < m)}
// ------------------------------------------------------------------------------------------
constexpr uint32_t kRankTile = 2048;

__global__ void __launch_bounds__(256)
k_rank(const float* __restrict__ fitness, uint32_t P, int32_t* __restrict__ rank,
       float* __restrict__ u, DeviceStatus* status)
{
    __shared__ float tile[kRankTile];
    dep_wait();
    dep_trigger();
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    const float fm = (m < P) ? fitness[m] : 0.f;
    if (m < P && fm != fm) atomicOr(&status->nonfinite, 1u);
    uint32_t below = 0;
    for (uint32_t base = 0; base < P; base += kRankTile) {
        const uint32_t n = min(kRankTile, P - base);
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) tile[i] = fitness[base + i];
        __syncthreads();
        if (m < P) {
            for (uint32_t i = 0; i < n; ++i) {
                const float fk = tile[i];
                below += (fk < fm || (fk == fm && base + i < m)) ? 1u : 0u;
            }
        }
    }
    if (m < P && EVO_IN_BOUNDS(status, EVO_SITE_RANK, m, P)) {
        rank[m] = static_cast<int32_t>(below);
        u[m] = __fadd_rn(__fdiv_rn(__uint2float_rn(below), __uint2float_rn(P - 1u)), -0.5f);
    }
}

// Larger populations: the comparisons of a member are split over blockIdx.y (one fitness tile of
// `tile_n` <= kRankTile entries each) and summed with integer atomics (exact, order-independent); a
// second kernel turns counts into centred ranks.
__global__ void __launch_bounds__(256)
k_rank_count(const float* __restrict__ fitness, uint32_t P, uint32_t tile_n, int32_t* __restrict__ rank,
             DeviceStatus* status)
{
    __shared__ float tile[kRankTile];
    dep_wait();
    dep_trigger();
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t base = blockIdx.y * tile_n;
    const uint32_t n = min(tile_n, P - base);
    for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) tile[i] = fitness[base + i];
    __syncthreads();
    if (m >= P) return;
    const float fm = fitness[m];
    if (blockIdx.y == 0 && fm != fm) atomicOr(&status->nonfinite, 1u);
    uint32_t below = 0;
#pragma unroll 8
    for (uint32_t i = 0; i < n; ++i) {
        const float fk = tile[i];
        below += (fk < fm || (fk == fm && base + i < m)) ? 1u : 0u;
    }
    atomicAdd(rank + m, static_cast<int32_t>(below));
}

__global__ void k_rank_zero(int32_t* __restrict__ rank, uint32_t P)
{
    dep_wait();
    dep_trigger();
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < P) rank[m] = 0;
}

__global__ void k_rank_finish(const int32_t* __restrict__ rank, uint32_t P, float* __restrict__ u)
{
    dep_wait();
    dep_trigger();
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < P)
        u[m] = __fadd_rn(__fdiv_rn(__uint2float_rn(static_cast<uint32_t>(rank[m])), __uint2float_rn(P - 1u)), -0.5f);
}

int launch_rank(cudaStream_t st, const float* fitness, uint32_t P, int32_t* rank, float* u,
                DeviceStatus* status)
{
    const uint32_t bx = (P + 255u) / 256u;
    if (P <= 1024u) {      // a handful of blocks, each thread against the whole population: a few microseconds
        return launch_dependent(k_rank, dim3(bx), dim3(256), 0, st, fitness, P, rank, u, status) == cudaSuccess ? 1 : -1;
    }
    // From there on one kernel of P / 256 blocks leaves most of the GPU idle (P = 4,096: 16 blocks, 63 us):
    // tiles of 256 comparisons up to P = 8,192 (P = 4,096: 256 blocks), of 2,048 beyond.
    const uint32_t tile_n = P <= 8192u ? 256u : kRankTile;
    if (launch_dependent(k_rank_zero, dim3(bx), dim3(256), 0, st, rank, P) != cudaSuccess) return -1;
    dim3 grid(bx, (P + tile_n - 1u) / tile_n);
    if (launch_dependent(k_rank_count, grid, dim3(256), 0, st, fitness, P, tile_n, rank, status) != cudaSuccess) return -1;
    return launch_dependent(k_rank_finish, dim3(bx), dim3(256), 0, st, rank, P, u) == cudaSuccess ? 3 : -1;
}

// ------------------------------------------------------------------------------------------
// ES gradient.  partial[s][d] = sum over the pairs of split s of (u[2j]-u[2j+1]) * eps[j][d],
// one thread per column quad.  Products and sums are fp64: the Adam step lr*g/(|g|+eps) is
// ill-conditioned where |g| is near adam_eps, so the cancellation error of an fp32 sum
// (~1e-7 of RMS(g)) would move those coordinates by far more than the 1e-5 parity bound.  The
// stored-noise kernel is HBM-bound (4 bytes per term), so the fp64 arithmetic is hidden.
// Summation order is fixed (two interleaved accumulators per column, splits added in order);
// no floating-point atomics anywhere, so results are run-to-run identical.
// REGEN recomputes eps from the Philox counters instead of reading it.
// ------------------------------------------------------------------------------------------
struct Acc4 { double x, y, z, w; };

__device__ __forceinline__ void acc_fma(Acc4& a, double wd, const float4& e)
{
    a.x = fma(wd, static_cast<double>(e.x), a.x);
    a.y = fma(wd, static_cast<double>(e.y), a.y);
    a.z = fma(wd, static_cast<double>(e.z), a.z);
    a.w = fma(wd, static_cast<double>(e.w), a.w);
}

constexpr int kGradThreads = 256;      // threads per block of the gradient kernel
constexpr int kGradRows = 4;           // noise rows in flight per thread (multiple of 2)

// SIGMA also accumulates the PGPE sigma gradient sum_j ((u[2j]+u[2j+1])/2) (eps^2 - 1) in fp32 (a plain
// step on sigma follows, which is not ill-conditioned like Adam's normalised step).
__device__ __forceinline__ void sig_fma(float4& a, float sj, const float4& e)
{
    a.x = fmaf(sj, fmaf(e.x, e.x, -1.0f), a.x);
    a.y = fmaf(sj, fmaf(e.y, e.y, -1.0f), a.y);
    a.z = fmaf(sj, fmaf(e.z, e.z, -1.0f), a.z);
    a.w = fmaf(sj, fmaf(e.w, e.w, -1.0f), a.w);
}

template <bool REGEN, bool SIGMA>
__global__ void __launch_bounds__(kGradThreads)
k_grad_partial(const float* __restrict__ u, const float* __restrict__ eps, PhiloxKey key,
               uint32_t pair0, uint32_t H, uint32_t D, uint32_t ldD,
               uint32_t pairs_per_split, double* __restrict__ partial, float* __restrict__ sigma_partial,
               const DeviceStatus* status)
{
    dep_wait();
    dep_trigger();
    if (status->nonfinite) return;
    const uint32_t quad = blockIdx.x * blockDim.x + threadIdx.x;
    if (quad * 4u >= ldD) return;
    const uint32_t generation = status->generation;
    const uint32_t j0 = blockIdx.y * pairs_per_split;
    const uint32_t j1 = min(H, j0 + pairs_per_split);
    Acc4 acc[2] = { {0., 0., 0., 0.}, {0., 0., 0., 0.} };
    float4 sacc[2] = { make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f) };
    const float2* up = reinterpret_cast<const float2*>(u) + pair0;    // u is global, eps rows are the shard's
    uint32_t j = j0;
    for (; j + kGradRows <= j1; j += kGradRows) {
        float4 e[kGradRows];
        double w[kGradRows];
        float sj[kGradRows];
#pragma unroll
        for (int i = 0; i < kGradRows; ++i) {
            if (REGEN) e[i] = stream_normal4(key, 0u, generation, pair0 + j + i, quad);
            else e[i] = __ldcs(reinterpret_cast<const float4*>(eps + static_cast<size_t>(j + i) * ldD) + quad);
            const float2 uu = __ldg(up + j + i);
            w[i] = static_cast<double>(uu.x) - static_cast<double>(uu.y);   // exact
            sj[i] = 0.5f * (uu.x + uu.y);
        }
#pragma unroll
        for (int i = 0; i < kGradRows; ++i) {
            acc_fma(acc[i & 1], w[i], e[i]);
            if (SIGMA) sig_fma(sacc[i & 1], sj[i], e[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < kGradRows - 1; ++i) {      // tail keeps the accumulator assignment j % 2
        if (j + i < j1) {
            float4 e;
            if (REGEN) e = stream_normal4(key, 0u, generation, pair0 + j + i, quad);
            else e = __ldcs(reinterpret_cast<const float4*>(eps + static_cast<size_t>(j + i) * ldD) + quad);
            const float2 uu = __ldg(up + j + i);
            acc_fma(acc[i & 1], static_cast<double>(uu.x) - static_cast<double>(uu.y), e);
            if (SIGMA) sig_fma(sacc[i & 1], 0.5f * (uu.x + uu.y), e);
        }
    }
    double r[4] = { acc[0].x + acc[1].x, acc[0].y + acc[1].y, acc[0].z + acc[1].z, acc[0].w + acc[1].w };
    if (REGEN && quad * 4u + 4u > D) {             // recomputed noise exists only for real columns
#pragma unroll
        for (uint32_t i = 0; i < 4u; ++i)
            if (quad * 4u + i >= D) r[i] = 0.;
    }
    double2* out = reinterpret_cast<double2*>(partial + static_cast<size_t>(blockIdx.y) * ldD) + 2u * quad;
    if (EVO_IN_BOUNDS(status, EVO_SITE_GRAD_PARTIAL, static_cast<size_t>(blockIdx.y) * ldD + 4u * quad + 3u,
                      static_cast<size_t>((H + pairs_per_split - 1u) / pairs_per_split) * ldD)) {
        out[0] = make_double2(r[0], r[1]);
        out[1] = make_double2(r[2], r[3]);
    }
    if (SIGMA) {
        float4 sr = make_float4(sacc[0].x + sacc[1].x, sacc[0].y + sacc[1].y, sacc[0].z + sacc[1].z, sacc[0].w + sacc[1].w);
        if (quad * 4u + 4u > D) {                  // padding columns carry no sigma signal
            if (quad * 4u + 0u >= D) sr.x = 0.f;
            if (quad * 4u + 1u >= D) sr.y = 0.f;
            if (quad * 4u + 2u >= D) sr.z = 0.f;
            if (quad * 4u + 3u >= D) sr.w = 0.f;
        }
        reinterpret_cast<float4*>(sigma_partial + static_cast<size_t>(blockIdx.y) * ldD)[quad] = sr;
    }
}

// Sum the splits in order, scale by sigma[d]/P, round the gradient to fp32; then either take the
// Adam ascent step (ADAM) or leave the step to the ClipUp kernels and emit this block's share of
// |g|^2; finally adapt sigma if a sigma gradient was accumulated.
template <bool ADAM>
__global__ void __launch_bounds__(256)
k_update(const double* __restrict__ partial, const float* __restrict__ sigma_partial, uint32_t splits,
         uint32_t ldD, double inv_pop, float lr, float beta1, float beta2, float adam_eps,
         float sigma_lr, float sigma_max_change, float inv_pairs, float* __restrict__ sigma_vec,
         float* __restrict__ center, float* __restrict__ m, float* __restrict__ v, float* __restrict__ g,
         double* __restrict__ norm_partial, const DeviceStatus* status)
{
    dep_wait();
    dep_trigger();
    if (status->nonfinite) return;
    __shared__ float corr[2];
    __shared__ double red[256];
    if (ADAM && threadIdx.x == 0) {
        const double t = static_cast<double>(status->adam_step + 1u);
        corr[0] = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta1), t)));
        corr[1] = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(beta2), t)));
    }
    __syncthreads();
    const uint32_t quad = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = quad * 4u < ldD;
    double gsq = 0.0;
    if (live) {
        double sum[4] = { 0., 0., 0., 0. };
        for (uint32_t k = 0; k < splits; ++k) {
            const double2* p = reinterpret_cast<const double2*>(partial + static_cast<size_t>(k) * ldD) + 2u * quad;
            const double2 a = p[0], b = p[1];
            sum[0] += a.x; sum[1] += a.y; sum[2] += b.x; sum[3] += b.y;
        }
        const float4 s4 = reinterpret_cast<const float4*>(sigma_vec)[quad];
        float sg[4] = { s4.x, s4.y, s4.z, s4.w };
        float gg[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            gg[i] = static_cast<float>(sum[i] * (static_cast<double>(sg[i]) * inv_pop));
            gsq += static_cast<double>(gg[i]) * static_cast<double>(gg[i]);
        }
        reinterpret_cast<float4*>(g)[quad] = make_float4(gg[0], gg[1], gg[2], gg[3]);
        if (ADAM) {
            float4 c4 = reinterpret_cast<float4*>(center)[quad];
            float4 m4 = reinterpret_cast<float4*>(m)[quad];
            float4 v4 = reinterpret_cast<float4*>(v)[quad];
            float cc[4] = { c4.x, c4.y, c4.z, c4.w }, mm[4] = { m4.x, m4.y, m4.z, m4.w },
                  vv[4] = { v4.x, v4.y, v4.z, v4.w };
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                mm[i] = beta1 * mm[i] + (1.f - beta1) * gg[i];
                vv[i] = beta2 * vv[i] + (1.f - beta2) * gg[i] * gg[i];
                const float mhat = mm[i] * corr[0];
                const float vhat = vv[i] * corr[1];
                cc[i] += lr * mhat / (sqrtf(vhat) + adam_eps);
            }
            reinterpret_cast<float4*>(m)[quad] = make_float4(mm[0], mm[1], mm[2], mm[3]);
            reinterpret_cast<float4*>(v)[quad] = make_float4(vv[0], vv[1], vv[2], vv[3]);
            if (EVO_IN_BOUNDS(status, EVO_SITE_UPDATE, 4u * quad + 3u, ldD))
                reinterpret_cast<float4*>(center)[quad] = make_float4(cc[0], cc[1], cc[2], cc[3]);
        }
        if (sigma_partial) {                            // PGPE sigma step with a relative-change limit
            float ss[4] = { 0.f, 0.f, 0.f, 0.f };
            for (uint32_t k = 0; k < splits; ++k) {
                const float4 p = reinterpret_cast<const float4*>(sigma_partial + static_cast<size_t>(k) * ldD)[quad];
                ss[0] += p.x; ss[1] += p.y; ss[2] += p.z; ss[3] += p.w;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float gs = sg[i] * inv_pairs * ss[i];
                const float lo = sg[i] * (1.f - sigma_max_change), hi = sg[i] * (1.f + sigma_max_change);
                sg[i] = fminf(fmaxf(sg[i] + sigma_lr * gs, lo), hi);
            }
            reinterpret_cast<float4*>(sigma_vec)[quad] = make_float4(sg[0], sg[1], sg[2], sg[3]);
        }
    }
    if (!ADAM) {                                        // fixed-order block sum of |g|^2
        red[threadIdx.x] = gsq;
        __syncthreads();
        for (uint32_t off = 128; off > 0; off >>= 1) {
            if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
            __syncthreads();
        }
        if (threadIdx.x == 0) norm_partial[blockIdx.x] = red[0];
    }
}

// ClipUp, step 1: vel = momentum vel + lr g/|g| and this block's share of |vel|^2.
// norm_partial: [0, nb) block sums of |g|^2 (in), [nb, 2nb) block sums of |vel|^2 (out).
__global__ void __launch_bounds__(256)
k_clipup_velocity(const float* __restrict__ g, float* __restrict__ vel, uint32_t ldD, float lr, float momentum,
                  double* __restrict__ norm_partial, uint32_t nb, const DeviceStatus* status)
{
    if (status->nonfinite) return;
    __shared__ double red[256];
    __shared__ float inv_gnorm;
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (uint32_t b = 0; b < nb; ++b) s += norm_partial[b];           // same order in every block
        inv_gnorm = s > 0.0 ? static_cast<float>(1.0 / sqrt(s)) : 0.f;
    }
    __syncthreads();
    const uint32_t quad = blockIdx.x * blockDim.x + threadIdx.x;
    double vsq = 0.0;
    if (quad * 4u < ldD) {
        const float4 g4 = reinterpret_cast<const float4*>(g)[quad];
        float4 v4 = reinterpret_cast<float4*>(vel)[quad];
        const float k = lr * inv_gnorm;
        v4.x = fmaf(momentum, v4.x, k * g4.x); v4.y = fmaf(momentum, v4.y, k * g4.y);
        v4.z = fmaf(momentum, v4.z, k * g4.z); v4.w = fmaf(momentum, v4.w, k * g4.w);
        reinterpret_cast<float4*>(vel)[quad] = v4;
        vsq = static_cast<double>(v4.x) * v4.x + static_cast<double>(v4.y) * v4.y +
              static_cast<double>(v4.z) * v4.z + static_cast<double>(v4.w) * v4.w;
    }
    red[threadIdx.x] = vsq;
    __syncthreads();
    for (uint32_t off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) norm_partial[nb + blockIdx.x] = red[0];
}

// ClipUp, step 2: clip |vel| to max_speed and move the centre.
__global__ void __launch_bounds__(256)
k_clipup_apply(float* __restrict__ vel, float* __restrict__ center, uint32_t ldD, float max_speed,
               const double* __restrict__ norm_partial, uint32_t nb, const DeviceStatus* status)
{
    if (status->nonfinite) return;
    __shared__ float scale;
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (uint32_t b = 0; b < nb; ++b) s += norm_partial[nb + b];
        const double vn = sqrt(s);
        scale = vn > static_cast<double>(max_speed) ? static_cast<float>(static_cast<double>(max_speed) / vn) : 1.0f;
    }
    __syncthreads();
    const uint32_t quad = blockIdx.x * blockDim.x + threadIdx.x;
    if (quad * 4u >= ldD) return;
    float4 v4 = reinterpret_cast<float4*>(vel)[quad];
    float4 c4 = reinterpret_cast<float4*>(center)[quad];
    v4.x *= scale; v4.y *= scale; v4.z *= scale; v4.w *= scale;
    c4.x += v4.x; c4.y += v4.y; c4.z += v4.z; c4.w += v4.w;
    reinterpret_cast<float4*>(vel)[quad] = v4;
    reinterpret_cast<float4*>(center)[quad] = c4;
}

// Closes a tell: the Adam step counter advances only if the update was applied; the generation
// counter (the random streams of the next ask and roll-out) always does.
__global__ void k_tell_finish(DeviceStatus* status)
{
    dep_wait();
    dep_trigger();
    if (status->nonfinite) {
        status->sticky |= (1u << EVO_ERR_NONFINITE);
        status->nonfinite = 0;
    } else {
        status->adam_step += 1u;
    }
    status->generation += 1u;
}

uint32_t gradient_splits(uint32_t H, uint32_t ldD)
{
    // enough thread blocks to fill 148 SMs several times over, a pure function of the shape
    const uint32_t blocks_x = (ldD / 4u + kGradThreads - 1u) / kGradThreads;
    uint32_t s = (148u * 32u + blocks_x - 1u) / blocks_x;
    if (s > 64u) s = 64u;
    const uint32_t max_s = (H + 15u) / 16u;            // at least 16 pairs per split
    if (s > max_s) s = max_s;
    if (s < 1u) s = 1u;
    return s;
}

size_t clipup_norm_doubles(uint32_t ldD) { return 2u * ((ldD / 4u + 255u) / 256u); }

template <bool REGEN, bool SIGMA>
static void launch_grad(dim3 grid, cudaStream_t st, const TellArgs& a, uint32_t pps)
{
    launch_dependent(k_grad_partial<REGEN, SIGMA>, grid, dim3(kGradThreads), 0, st, a.u, a.eps, philox_key(a.k0, a.k1),
                     a.pair0, a.H, a.D, a.ldD, pps, a.partial, a.sigma_partial, a.status);
}

static int launch_partials(cudaStream_t st, const TellArgs& a, uint32_t* used_out)
{
    const uint32_t quads = a.ldD / 4u;
    const uint32_t pps = (a.H + a.splits - 1u) / a.splits;
    const uint32_t used = (a.H + pps - 1u) / pps;      // splits that own at least one pair
    dim3 grid((quads + kGradThreads - 1u) / kGradThreads, used);
    const bool sig = a.sigma_partial != nullptr;
    if (a.eps) { if (sig) launch_grad<false, true>(grid, st, a, pps); else launch_grad<false, false>(grid, st, a, pps); }
    else       { if (sig) launch_grad<true, true>(grid, st, a, pps);  else launch_grad<true, false>(grid, st, a, pps); }
    *used_out = used;
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// optimiser step (and sigma step) from `splits` rows of partial sums
static int launch_step(cudaStream_t st, const TellArgs& a, const double* partial, const float* sigma_partial,
                       uint32_t splits)
{
    const uint32_t quads = a.ldD / 4u;
    const double inv_pop = 1.0 / static_cast<double>(a.P);
    const float inv_pairs = 2.0f / static_cast<float>(a.P);
    const uint32_t nb = (quads + 255u) / 256u;
    int launches = 0;
    if (a.optimizer == EVO_OPT_ADAM) {
        if (launch_dependent(k_update<true>, dim3(nb), dim3(256), 0, st, partial, sigma_partial, splits, a.ldD, inv_pop, a.lr,
                             a.beta1, a.beta2, a.adam_eps, a.sigma_lr, a.sigma_max_change, inv_pairs, a.sigma_vec,
                             a.center, a.m, a.v, a.g, a.norms, a.status) != cudaSuccess) return -1;
        launches += 1;
    } else {
        if (launch_dependent(k_update<false>, dim3(nb), dim3(256), 0, st, partial, sigma_partial, splits, a.ldD, inv_pop, a.lr,
                             a.beta1, a.beta2, a.adam_eps, a.sigma_lr, a.sigma_max_change, inv_pairs, a.sigma_vec,
                             a.center, a.m, a.v, a.g, a.norms, a.status) != cudaSuccess) return -1;
        k_clipup_velocity<<<nb, 256, 0, st>>>(a.g, a.m, a.ldD, a.lr, a.clipup_momentum, a.norms, nb, a.status);
        if (cudaGetLastError() != cudaSuccess) return -1;
        k_clipup_apply<<<nb, 256, 0, st>>>(a.m, a.center, a.ldD, a.clipup_max_speed, a.norms, nb, a.status);
        if (cudaGetLastError() != cudaSuccess) return -1;
        launches += 3;
    }
    if (launch_dependent(k_tell_finish, dim3(1), dim3(1), 0, st, a.status) != cudaSuccess) return -1;
    return launches + 1;
}

int launch_gradient_update(cudaStream_t st, const TellArgs& a)
{
    uint32_t used = 0;
    const int n1 = launch_partials(st, a, &used);
    if (n1 < 0) return -1;
    const int n2 = launch_step(st, a, a.partial, a.sigma_partial, used);
    return n2 < 0 ? -1 : n1 + n2;
}

// splits -> one row each, in split order (the buffers the caller sums across shards); a skipped
// update (NaN fitness) leaves zeros so that the all-reduce still runs on defined values
__global__ void __launch_bounds__(256)
k_sum_splits(const double* __restrict__ partial, const float* __restrict__ sigma_partial, uint32_t splits,
             uint32_t ldD, double* __restrict__ grad_sum, float* __restrict__ sigma_sum, const DeviceStatus* status)
{
    const uint32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= ldD) return;
    const bool skip = status->nonfinite != 0;
    double s = 0.0;
    float t = 0.f;
    if (!skip) {
        for (uint32_t k = 0; k < splits; ++k) s += partial[static_cast<size_t>(k) * ldD + d];
        if (sigma_partial)
            for (uint32_t k = 0; k < splits; ++k) t += sigma_partial[static_cast<size_t>(k) * ldD + d];
    }
    grad_sum[d] = s;
    if (sigma_sum) sigma_sum[d] = t;
}

int launch_gradient_sums(cudaStream_t st, const TellArgs& a, double* grad_sum, float* sigma_sum)
{
    uint32_t used = 0;
    if (launch_partials(st, a, &used) < 0) return -1;
    k_sum_splits<<<(a.ldD + 255u) / 256u, 256, 0, st>>>(a.partial, a.sigma_partial, used, a.ldD, grad_sum,
                                                        a.sigma_partial ? sigma_sum : nullptr, a.status);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

int launch_update_from_sums(cudaStream_t st, const TellArgs& a, const double* grad_sum, const float* sigma_sum)
{
    return launch_step(st, a, grad_sum, a.sigma_partial ? sigma_sum : nullptr, 1u);
}

}  // namespace evo
