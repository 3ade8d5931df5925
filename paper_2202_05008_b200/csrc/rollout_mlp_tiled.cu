// Fast control-task rollout for compile-time network shapes.
//
// Block = (member, block of EB episodes).  The member's parameter row is fetched from HBM once
// with a single bulk asynchronous copy (cp.async.bulk, completion on an mbarrier), then every
// thread moves its slice of each weight matrix into REGISTERS, where it stays for all T steps:
// the FP32 pipe needs one operand per FMA from somewhere, and shared memory (128 B/clk/SM) can
// feed only a quarter of the 128 FMA lanes, so weights live in registers and only the small
// activation vectors ([unit][episode], a few hundred bytes) travel through shared memory as
// broadcast 128-bit loads.  A thread owns TI output rows x KS inputs of a layer (inputs s, s+S,
// s+2S, ... so that the S lanes read adjacent shared-memory words); the S threads
// that share a row group are adjacent lanes and combine their partial sums with shuffles.
// Task state stays in registers / shared memory; nothing but the optional debug trace and one
// partial return per block goes back to HBM.
//
// Paper: Section 2 (roll-out loop, central seeds), Section 4 (get_actions over the population
// with parameters as data; stateless task step; identical initial observations).
#include "internal.h"
#include "async.cuh"
#include "fp32x2.cuh"
#include "noise.cuh"
#include "tasks.cuh"

namespace evo {

// tanh(x) = 1 - 2/(exp(2x)+1) on the special-function unit; absolute error ~2e-7
__device__ __forceinline__ float tanh_fast(float x)
{
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 2.885390082f));      // e^(2x) = 2^(2x log2 e)
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.0f));
    return fmaf(-2.0f, r, 1.0f);
}

template <int EB> struct EpVec;
template <> struct EpVec<1> { static __device__ __forceinline__ void load(const float* p, float* a) { a[0] = p[0]; } };
template <> struct EpVec<2> { static __device__ __forceinline__ void load(const float* p, float* a) {
    const float2 v = *reinterpret_cast<const float2*>(p); a[0] = v.x; a[1] = v.y; } };
template <> struct EpVec<4> { static __device__ __forceinline__ void load(const float* p, float* a) {
    const float4 v = *reinterpret_cast<const float4*>(p); a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w; } };
template <> struct EpVec<8> { static __device__ __forceinline__ void load(const float* p, float* a) {
    const float4 v = reinterpret_cast<const float4*>(p)[0], u = reinterpret_cast<const float4*>(p)[1];
    a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w; a[4] = u.x; a[5] = u.y; a[6] = u.z; a[7] = u.w; } };
template <> struct EpVec<16> { static __device__ __forceinline__ void load(const float* p, float* a) {
    EpVec<8>::load(p, a); EpVec<8>::load(p + 8, a + 8); } };

__host__ __device__ constexpr int ilog2(int x) { return x <= 1 ? 0 : 1 + ilog2(x / 2); }

// Sum v[0..N) over the S adjacent lanes that share a row group.  While more than one value is
// left each stage halves the set a lane keeps (lanes exchange the halves they give up); after
// that the remaining stages are plain butterflies.  On return the lane holds CNT = max(N/S, 1)
// finished sums, v[0..CNT), belonging to indices [offset, offset + CNT).
template <int N, int S>
__device__ __forceinline__ int reduce_lanes(float (&v)[N], int s)
{
    int offset = 0;
    int cur = N;
#pragma unroll
    for (int b = 0; b < ilog2(S); ++b) {
        const bool upper = (s >> b) & 1;
        if (cur > 1) {
            const int half = cur / 2;
#pragma unroll
            for (int i = 0; i < N / 2; ++i) {
                if (i < half) {
                    const float keep = upper ? v[half + i] : v[i];
                    const float give = upper ? v[i] : v[half + i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, give, 1 << b);
                }
            }
            if (upper) offset += half;
            cur = half;
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1 << b);
        }
    }
    return offset;
}

// Select-free variant for TI >= S: register slot i of lane s holds output row i ^ rowmask(s) with
// rowmask(s) = sum_b bit_b(s) * (TI >> (b+1)), so at every stage a lane keeps its lower slots and
// hands over its upper ones.  Returns rowmask(s): the lane ends with rows rowmask(s) .. + TI/S - 1.
template <int S> __device__ __forceinline__ int row_mask(int s, int TI)
{
    int m = 0;
#pragma unroll
    for (int b = 0; b < ilog2(S); ++b) m += ((s >> b) & 1) * (TI >> (b + 1));
    return m;
}

template <int TI, int EB, int S>
__device__ __forceinline__ void reduce_lanes_perm(float (&v)[TI * EB])
{
#pragma unroll
    for (int b = 0; b < ilog2(S); ++b) {
        const int half = TI >> (b + 1);
#pragma unroll
        for (int i = 0; i < TI / 2; ++i) {
            if (i < half) {
#pragma unroll
                for (int e = 0; e < EB; ++e)
                    v[i * EB + e] += __shfl_xor_sync(0xffffffffu, v[(half + i) * EB + e], 1 << b);
            }
        }
    }
}

// One dense layer y = f(W x + b) for EB episodes at once.
//   NI inputs, NO outputs, thread tile TI rows x KS = NI/S inputs, S lanes per row group.
//   LD = floats between consecutive units of the activation arrays (>= EB; a team that owns only
//   some of the episodes of a wider array passes the array's full episode count).
template <int NI, int NO, int TI, int S, int EB, int THREADS, int LD = EB>
struct Dense {
    static_assert(NI % S == 0, "S must divide the input width");
    static_assert((S & (S - 1)) == 0 && S <= 32, "S is a power of two within a warp");
    static constexpr int KS = NI / S;
    static constexpr int GROUPS = (NO + TI - 1) / TI;
    static constexpr int ACTIVE = GROUPS * S;
    static_assert(ACTIVE <= THREADS, "layer needs more threads than the block has");
    static constexpr int N = TI * EB;
    static constexpr int CNT = (N >= S) ? N / S : 1;
    static constexpr bool PERM = (TI >= S) && (S > 1);        // select-free reduction possible

    float w[TI][KS];
    float bias[TI];
    int   row0, s;
    bool  active;

    // weights from a row-major [no][ni] matrix followed by bias[no] (shared or global memory).  The
    // layer may be narrower than the compiled tile (no <= NO, ni <= NI): the missing rows and columns
    // are zeros, so the padded units are tanh(0) = 0 and feed nothing into the next layer.
    __device__ __forceinline__ void load(const float* W, const float* b, int tid, int ni = NI, int no = NO)
    {
        active = tid < ACTIVE;
        s = tid % S;
        row0 = (tid / S) * TI;
        const int rm = PERM ? row_mask<S>(s, TI) : 0;
#pragma unroll
        for (int r = 0; r < TI; ++r) {
            const int row = row0 + (r ^ rm);                     // slot r holds this output row
            const bool ok = active && (row < no);
#pragma unroll
            for (int k = 0; k < KS; ++k) w[r][k] = (ok && k * S + s < ni) ? W[row * ni + k * S + s] : 0.f;
            bias[r] = (ok && s == 0 && b) ? b[row] : 0.f;
        }
    }

    // in: [NI][EB], out: [NO][EB]; out = scale * tanh(.) if ACT else the plain sum
    template <bool ACT, class Hook>
    __device__ __forceinline__ void run(const float* __restrict__ in, float* __restrict__ out,
                                        float scale, Hook&& hook) const
    {
        float acc[N];
        if constexpr (TI % 2 == 0) {
            // rows in pairs: one paired FMA updates rows 2j and 2j+1 of an episode
            float2 acc2[TI / 2][EB];
#pragma unroll
            for (int j = 0; j < TI / 2; ++j)
#pragma unroll
                for (int e = 0; e < EB; ++e) acc2[j][e] = make_float2(bias[2 * j], bias[2 * j + 1]);
#pragma unroll
            for (int k = 0; k < KS; ++k) {
                float a[EB];
                EpVec<EB>::load(in + (k * S + s) * LD, a);     // lane s takes inputs s, s+S, ... (no bank conflicts)
                hook(k * S + s, a);
#pragma unroll
                for (int e = 0; e < EB; ++e) {
                    const float2 aa = make_float2(a[e], a[e]);
#pragma unroll
                    for (int j = 0; j < TI / 2; ++j) ffma2(acc2[j][e], make_float2(w[2 * j][k], w[2 * j + 1][k]), aa);
                }
            }
#pragma unroll
            for (int j = 0; j < TI / 2; ++j)
#pragma unroll
                for (int e = 0; e < EB; ++e) { acc[(2 * j) * EB + e] = acc2[j][e].x; acc[(2 * j + 1) * EB + e] = acc2[j][e].y; }
        } else {
#pragma unroll
            for (int r = 0; r < TI; ++r)
#pragma unroll
                for (int e = 0; e < EB; ++e) acc[r * EB + e] = bias[r];
#pragma unroll
            for (int k = 0; k < KS; ++k) {
                float a[EB];
                EpVec<EB>::load(in + (k * S + s) * LD, a);     // lane s takes inputs s, s+S, ... (no bank conflicts)
                hook(k * S + s, a);
#pragma unroll
                for (int r = 0; r < TI; ++r)
#pragma unroll
                    for (int e = 0; e < EB; ++e) acc[r * EB + e] = fmaf(w[r][k], a[e], acc[r * EB + e]);
            }
        }
        int offset;
        if constexpr (PERM) { reduce_lanes_perm<TI, EB, S>(acc); offset = row_mask<S>(s, TI) * EB; }
        else offset = reduce_lanes<N, S>(acc, s);
        // with N < S several lanes end with the same sum: the one whose spare bits are 0 writes
        const bool writer = active && ((N >= S) || ((s >> ilog2(N)) == 0));
        if (writer) {
            if constexpr (CNT >= EB && EB >= 4) {              // whole rows: 128-bit stores
#pragma unroll
                for (int i = 0; i < CNT; i += 4) {
                    const int n = offset + i;
                    const int row = row0 + n / EB, e = n % EB;
                    float4 y;
                    y.x = ACT ? scale * tanh_fast(acc[i + 0]) : acc[i + 0];
                    y.y = ACT ? scale * tanh_fast(acc[i + 1]) : acc[i + 1];
                    y.z = ACT ? scale * tanh_fast(acc[i + 2]) : acc[i + 2];
                    y.w = ACT ? scale * tanh_fast(acc[i + 3]) : acc[i + 3];
                    if (row < NO) *reinterpret_cast<float4*>(out + row * LD + e) = y;
                }
            } else {
#pragma unroll
                for (int i = 0; i < CNT; ++i) {
                    const int n = offset + i;
                    const int row = row0 + n / EB, e = n % EB;
                    if (row < NO) out[row * LD + e] = ACT ? scale * tanh_fast(acc[i]) : acc[i];
                }
            }
        }
    }
};

struct NoHook { __device__ __forceinline__ void operator()(int, const float*) const {} };

template <int NIN, int H1, int H2, int NOUT, int EB, int THREADS, int TASK,
          int TI1, int S1, int TI2, int S2, int TI3, int S3>
__global__ void __launch_bounds__(THREADS)
k_rollout_mlp_tiled(const RolloutMlpArgs a, DeviceStatus* status)
{
    dep_wait();
    constexpr bool CART = (TASK == EVO_TASK_CARTPOLE);
    constexpr int NOBS = CART ? 5 : (kTlNx + kTlNa);        // tanh-linear: [x ; a] feeds the dynamics
    static_assert(!CART || S3 * ((NOUT + TI3 - 1) / TI3) <= 32, "cart-pole action layer runs in warp 0");
    static_assert(CART ? (NIN == 5 && NOUT == 1) : (NIN == kTlNx && NOUT == kTlNa), "task/policy shape");

    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) uint64_t mbar;
    float* stage = smem;                                      // parameter row, ldD floats
    float* obs0 = stage + a.ldD;                              // [NOBS][EB]
    float* obs1 = obs0 + NOBS * EB;                           // second x buffer (tanh-linear)
    float* h1 = obs1 + NOBS * EB;                             // [H1][EB]
    float* h2 = h1 + H1 * EB;                                 // [H2][EB]
    float* actb = h2 + H2 * EB;                               // [NOUT][EB] (cart-pole)

    const int tid = threadIdx.x;
    const uint32_t member = blockIdx.x, eb = blockIdx.y;
    const uint32_t e0 = eb * EB;
    const int nE = min(static_cast<uint32_t>(EB), a.E - e0);
    const PhiloxKey key = philox_key(a.k0, a.k1);

    // ---- parameter row: one bulk copy HBM -> shared memory ---------------------------------
    const uint32_t bar = smem_u32(&mbar);
    if (tid == 0) { mbar_init(bar, 1); mbar_init_fence(); }
    __syncthreads();
    if (tid == 0 && !(status->debug_flags & EVO_DEBUG_DROP_COMPLETION))   // the member's whole parameter row in one bulk copy
        bulk_copy_g2s(smem_u32(stage), a.theta + static_cast<size_t>(member) * a.ldD, a.ldD * 4u, bar);

    // ---- reset (overlaps the copy) -----------------------------------------------------------
    CartpoleConst cpc{};
    CpState cps{};
    float snc = 0.f, csc = 1.f;             // sin/cos of the pole angle, carried from the observation
    float ret = 0.f;                        // cart-pole: lane e of warp 0; tanh-linear: see below
    if (CART) {
        cpc = cartpole_const(a.tp);
        if (tid < EB) {
            cps = cartpole_reset(key, status->generation, e0 + min(tid, nE - 1), a.tp[EVO_CP_INIT_RANGE]);
            float sn, cs;
            sincos_fast(cps.th, sn, cs);
            snc = sn; csc = cs;
            obs0[0 * EB + tid] = cps.x;  obs0[1 * EB + tid] = cps.xd;
            obs0[2 * EB + tid] = cs;     obs0[3 * EB + tid] = sn;
            obs0[4 * EB + tid] = cps.thd;
        }
    } else {
        for (int item = tid; item < (kTlNx / 4) * EB; item += THREADS) {
            const int q = item / EB, e = item % EB;
            const float4 z = stream_normal4(key, 1u, status->generation, e0 + min(e, nE - 1), q);
            obs0[(4 * q + 0) * EB + e] = z.x; obs0[(4 * q + 1) * EB + e] = z.y;
            obs0[(4 * q + 2) * EB + e] = z.z; obs0[(4 * q + 3) * EB + e] = z.w;
        }
    }

    // one thread waits (bounded) and publishes the outcome, so the whole block takes one branch
    __shared__ int copy_ok;
    if (tid == 0) {
        copy_ok = mbar_wait_bounded(bar, 0u, &status->wait_cycles_log2) ? 1 : 0;
        if (!copy_ok) {
            // the copy did not land in time: flag it, give it one more bounded chance (so that it is
            // not still writing into shared memory that the next block gets), and leave a NaN as
            // this block's return: the member's fitness is then NaN and tell skips the update
            atomicOr(&status->sticky, 1u << EVO_ERR_TIMEOUT);
            mbar_wait_bounded(bar, 0u, &status->wait_cycles_log2);
            a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = __int_as_float(0x7FC00000);
        }
    }
    __syncthreads();
    if (!copy_ok) return;

    // ---- weights into registers ----------------------------------------------------------------
    Dense<NIN, H1, TI1, S1, EB, THREADS> L1;
    Dense<H1, H2, TI2, S2, EB, THREADS> L2;
    Dense<H2, NOUT, TI3, S3, EB, THREADS> L3;
    {
        const int n1 = static_cast<int>(a.sizes[1]), n2 = static_cast<int>(a.sizes[2]);   // real widths <= H1, H2
        const float* p = stage;
        L1.load(p, p + n1 * NIN, tid, NIN, n1); p += n1 * NIN + n1;
        L2.load(p, p + n2 * n1, tid, n1, n2);   p += n2 * n1 + n2;
        L3.load(p, p + NOUT * n2, tid, n2, NOUT);
    }
    // tanh-linear dynamics x' = tanh([A B][x ; a]) as a fourth layer with shared weights
    constexpr int SD = CART ? 1 : 4;
    constexpr int NID = CART ? 1 : NOBS, NOD = CART ? 1 : kTlNx;
    Dense<NID, NOD, 1, SD, EB, THREADS> LD;
    if (!CART) {
        LD.active = tid < LD.ACTIVE; LD.s = tid % SD; LD.row0 = tid / SD; LD.bias[0] = 0.f;
        const bool ok = LD.active && LD.row0 < NOD;
#pragma unroll
        for (int k = 0; k < LD.KS; ++k) {
            const int col = k * SD + LD.s;
            const float* A = a.task_const;
            const float* B = a.task_const + kTlNx * kTlNx;
            LD.w[0][k] = !ok ? 0.f : (col < static_cast<int>(kTlNx) ? A[LD.row0 * kTlNx + col]
                                                                    : B[LD.row0 * kTlNa + (col - kTlNx)]);
        }
    }
    __syncthreads();

    float* obs = obs0;
    float* obs_next = obs1;
    const bool tracing = a.trace != nullptr;

    // ---- time loop -------------------------------------------------------------------------------
    for (uint32_t t = 0; t < a.T; ++t) {
        L1.template run<true>(obs, h1, 1.0f, NoHook{});
        __syncthreads();
        L2.template run<true>(h1, h2, 1.0f, NoHook{});
        __syncthreads();
        if constexpr (CART) {
            // the action and the task step are one warp's work: no block-wide barrier in between
            if (tid < 32) {
                L3.template run<true>(h2, actb, a.action_scale, NoHook{});
                __syncwarp();
                if (tid < EB) {
                    cps = cartpole_step_fast_sc(cpc, cps, actb[tid], snc, csc);
                    float sn, cs;
                    sincos_fast(cps.th, sn, cs);
                    snc = sn; csc = cs;
                    ret += cs * __expf(-cps.x * cps.x);       // reward on the post-step state
                    obs[0 * EB + tid] = cps.x;  obs[1 * EB + tid] = cps.xd;
                    obs[2 * EB + tid] = cs;     obs[3 * EB + tid] = sn;
                    obs[4 * EB + tid] = cps.thd;
                    if (tracing && t < a.trace_T && tid < nE) {
                        float4* tr = reinterpret_cast<float4*>(
                            a.trace + ((static_cast<size_t>(member) * a.E + e0 + tid) * a.trace_T + t) * 4);
                        *tr = make_float4(cps.x, cps.xd, cps.th, cps.thd);
                    }
                }
            }
            __syncthreads();
        } else {
            // actions go straight behind x so that [x ; a] is one input vector of the dynamics
            L3.template run<true>(h2, obs + kTlNx * EB, a.action_scale, NoHook{});
            __syncthreads();
            // reward -|x|^2 - 0.01|a|^2 on (x_t, a_t): the S lanes of row group 0 see every input.
            // Squares of states and of actions are summed apart (which of the two an input slice
            // belongs to is known at compile time), two episodes per paired FMA.
            static_assert(EB == 4 && kTlNx % SD == 0, "reward sums are written for 4 episodes");
            float2 sx01 = make_float2(0.f, 0.f), sx23 = sx01, sa01 = sx01, sa23 = sx01;
            const bool group0 = tid < SD;
            LD.template run<true>(obs, obs_next, 1.0f, [&](int col, const float* v) {
                if (group0) {
                    const float2 v01 = make_float2(v[0], v[1]), v23 = make_float2(v[2], v[3]);
                    if (col - LD.s < static_cast<int>(kTlNx)) { ffma2(sx01, v01, v01); ffma2(sx23, v23, v23); }
                    else                                      { ffma2(sa01, v01, v01); ffma2(sa23, v23, v23); }
                }
            });
            if (tid < SD) {                                    // row group 0, whole warp-converged
                const float sq[4] = { fmaf(-0.01f, sa01.x, -sx01.x), fmaf(-0.01f, sa01.y, -sx01.y),
                                      fmaf(-0.01f, sa23.x, -sx23.x), fmaf(-0.01f, sa23.y, -sx23.y) };
#pragma unroll
                for (int e = 0; e < EB; ++e) if (e < nE) ret += sq[e];
            }
            if (tracing && t < a.trace_T) {
                __syncthreads();
                for (int item = tid; item < static_cast<int>(kTlNx) * nE; item += THREADS) {
                    const int i = item / nE, e = item % nE;
                    a.trace[((static_cast<size_t>(member) * a.E + e0 + e) * a.trace_T + t) * kTlNx + i] =
                        obs_next[i * EB + e];
                }
            }
            __syncthreads();
            float* tmp = obs; obs = obs_next; obs_next = tmp;
        }
    }

    // ---- block return: fixed-order sum over the block's episodes ---------------------------------
    if (tid < 32) {
        float v;
        if (CART) v = (tid < nE) ? ret : 0.f;
        else      v = (tid < SD) ? ret : 0.f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (tid == 0 && EVO_IN_BOUNDS(status, EVO_SITE_FIT_PARTIAL, static_cast<size_t>(member) * a.n_eb + eb,
                                      static_cast<size_t>(a.P) * a.n_eb))
            a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = v;
    }
}

// ------------------------------------------------------------------------------------------
// Cart-pole, warp-specialised: the task step (action layer + RK4, ~1 us of dependent latency on
// a handful of lanes) and the two wide policy layers take about equally long, so a block carries
// two groups of EB episodes and runs them half a step apart: while the task warp advances group
// A, the policy warps compute the hidden layers of group B, and vice versa.  Block = (member,
// 2*EB episodes); warp 0 = task warp; the policy warps form NT teams of MT threads, each team
// owning EB/NT episodes of the group (the weights are replicated in each team's registers).
// ------------------------------------------------------------------------------------------
template <int H1, int H2, int EB, int MT, int NT, int TI1, int S1, int TI2, int S2, int TI3, int S3>
__global__ void __launch_bounds__(32 + MT * NT)
k_rollout_cartpole_ws(const RolloutMlpArgs a, DeviceStatus* status)
{
    dep_wait();
    constexpr int NIN = 5;
    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) uint64_t mbar;
    __shared__ int copy_ok;
    float* stage = smem;                                   // parameter row
    float* obs = stage + a.ldD;                            // [2][NIN][EB]
    float* h1 = obs + 2 * NIN * EB;                        // [H1][EB]   (policy warps only)
    float* h2 = h1 + H1 * EB;                              // [2][H2][EB]

    const int tid = threadIdx.x;
    const uint32_t member = blockIdx.x, eb = blockIdx.y;
    const uint32_t e0 = eb * (2 * EB);
    const int nE = min(static_cast<uint32_t>(2 * EB), a.E - e0);      // episodes of this block
    const int nA = min(nE, EB), nB = nE - nA;                        // group sizes
    const PhiloxKey key = philox_key(a.k0, a.k1);

    const uint32_t bar = smem_u32(&mbar);
    if (tid == 0) { mbar_init(bar, 1); mbar_init_fence(); }
    __syncthreads();
    if (tid == 0 && !(status->debug_flags & EVO_DEBUG_DROP_COMPLETION))   // the member's whole parameter row in one bulk copy
        bulk_copy_g2s(smem_u32(stage), a.theta + static_cast<size_t>(member) * a.ldD, a.ldD * 4u, bar);
    // seeded starts of both groups (lanes e < EB of the task warp keep the states in registers)
    const CartpoleConst cpc = cartpole_const(a.tp);
    CpState cps[2] = {};
    float snc[2] = { 0.f, 0.f }, csc[2] = { 1.f, 1.f };    // sin/cos of the pole angle, carried from the observation
    float ret[2] = { 0.f, 0.f };
    if (tid < EB) {
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const int ng = g ? nB : nA;
            const uint32_t ep = e0 + g * EB + min(tid, max(ng, 1) - 1);
            cps[g] = cartpole_reset(key, status->generation, min(ep, a.E - 1u), a.tp[EVO_CP_INIT_RANGE]);
            float sn, cs;
            sincos_fast(cps[g].th, sn, cs);
            snc[g] = sn; csc[g] = cs;
            float* o = obs + g * NIN * EB;
            o[0 * EB + tid] = cps[g].x;  o[1 * EB + tid] = cps[g].xd;
            o[2 * EB + tid] = cs;        o[3 * EB + tid] = sn;
            o[4 * EB + tid] = cps[g].thd;
        }
    }
    if (tid == 0) {
        copy_ok = mbar_wait_bounded(bar, 0u, &status->wait_cycles_log2) ? 1 : 0;
        if (!copy_ok) {                                   // as in k_rollout_mlp_tiled
            atomicOr(&status->sticky, 1u << EVO_ERR_TIMEOUT);
            mbar_wait_bounded(bar, 0u, &status->wait_cycles_log2);
            a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = __int_as_float(0x7FC00000);
        }
    }
    __syncthreads();
    if (!copy_ok) return;

    const bool tracing = a.trace != nullptr;
    const int n1 = static_cast<int>(a.sizes[1]), n2 = static_cast<int>(a.sizes[2]);       // real widths <= H1, H2
    const float* p1 = stage;
    const float* p2 = p1 + n1 * NIN + n1;
    const float* p3 = p2 + n2 * n1 + n2;

    if (tid >= 32) {
        // ---------------- policy warps: hidden layers of one group per half step ----------------
        constexpr int ET = EB / NT;                        // episodes per team
        static_assert(EB % NT == 0, "teams split the group's episodes evenly");
        const int team = (tid - 32) / MT, mt = (tid - 32) % MT;
        const int eoff = team * ET;
        Dense<NIN, H1, TI1, S1, ET, MT, EB> L1;
        Dense<H1, H2, TI2, S2, ET, MT, EB> L2;
        L1.load(p1, p1 + n1 * NIN, mt, NIN, n1);
        L2.load(p2, p2 + n2 * n1, mt, n1, n2);
        auto hidden = [&](int g) {
            L1.template run<true>(obs + g * NIN * EB + eoff, h1 + eoff, 1.0f, NoHook{});
            asm volatile("bar.sync %0, %1;" :: "r"(1 + team), "n"(MT) : "memory");   // the team's own barrier
            L2.template run<true>(h1 + eoff, h2 + g * H2 * EB + eoff, 1.0f, NoHook{});
        };
        __syncthreads();                                   // weights are in registers everywhere
        hidden(0);
        __syncthreads();
        for (uint32_t t = 0; t < a.T; ++t) {
            hidden(1);
            __syncthreads();
            if (t + 1u < a.T) hidden(0);
            __syncthreads();
        }
    } else {
        // ---------------- task warp: action layer + RK4 step of the other group ------------------
        // action layer H2 -> 1: lane = (episode e = lane % EB, input slice q = lane / EB); every lane
        // ends with its episode's action after log2(32/EB) butterfly stages, no shared-memory trip
        constexpr int Q = 32 / EB, KQ = H2 / Q;
        static_assert(32 % EB == 0 && H2 % Q == 0, "action layer mapping");
        const int le = tid % EB, lq = tid / EB;
        float w3[KQ];
#pragma unroll
        for (int i = 0; i < KQ; ++i) w3[i] = (lq + Q * i < n2) ? p3[lq + Q * i] : 0.f;
        const float b3 = p3[n2];
        auto advance = [&](int g, uint32_t t) {
            const float* hin = h2 + g * H2 * EB;
            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
            for (int i = 0; i < KQ; i += 2) {
                acc0 = fmaf(w3[i], hin[(lq + Q * i) * EB + le], acc0);
                acc1 = fmaf(w3[i + 1], hin[(lq + Q * (i + 1)) * EB + le], acc1);
            }
            float pre = acc0 + acc1;
#pragma unroll
            for (int off = EB; off < 32; off <<= 1) pre += __shfl_xor_sync(0xffffffffu, pre, off);
            const float force = a.action_scale * tanh_fast(pre + b3);
            if (tid < EB) {
                cps[g] = cartpole_step_fast_sc(cpc, cps[g], force, snc[g], csc[g]);
                float sn, cs;
                sincos_fast(cps[g].th, sn, cs);
                snc[g] = sn; csc[g] = cs;
                ret[g] += cs * __expf(-cps[g].x * cps[g].x);       // reward on the post-step state
                float* o = obs + g * NIN * EB;
                o[0 * EB + tid] = cps[g].x;  o[1 * EB + tid] = cps[g].xd;
                o[2 * EB + tid] = cs;        o[3 * EB + tid] = sn;
                o[4 * EB + tid] = cps[g].thd;
                if (tracing && t < a.trace_T && tid < (g ? nB : nA)) {
                    float4* tr = reinterpret_cast<float4*>(
                        a.trace + ((static_cast<size_t>(member) * a.E + e0 + g * EB + tid) * a.trace_T + t) * 4);
                    *tr = make_float4(cps[g].x, cps[g].xd, cps[g].th, cps[g].thd);
                }
            }
            __syncwarp();
        };
        __syncthreads();
        __syncthreads();
        for (uint32_t t = 0; t < a.T; ++t) {
            advance(0, t);
            __syncthreads();
            advance(1, t);
            __syncthreads();
        }
        // block return: group A's episodes then group B's, butterfly sum (fixed order)
        float v = ((tid < nA) ? ret[0] : 0.f) + ((tid < nB) ? ret[1] : 0.f);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (tid == 0 && EVO_IN_BOUNDS(status, EVO_SITE_FIT_PARTIAL, static_cast<size_t>(member) * a.n_eb + eb,
                                      static_cast<size_t>(a.P) * a.n_eb))
            a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = v;
    }
}

// ------------------------------------------------------------------------------------------
// shapes with a compiled kernel
// ------------------------------------------------------------------------------------------
struct TiledShape { uint32_t task, nin, h1, h2, nout, EB; };
static const TiledShape kShapes[] = {
    { EVO_TASK_CARTPOLE, 5, 16, 16, 1, 1 },
    { EVO_TASK_CARTPOLE, 5, 64, 64, 1, 8 },
    { EVO_TASK_TANH_LINEAR, 28, 128, 128, 8, 4 },
    { EVO_TASK_CARTPOLE, 5, 32, 32, 1, 8 },
    { EVO_TASK_CARTPOLE, 5, 128, 128, 1, 8 },
};
static bool has_two_group_kernel(int shape) { return shape == 1 || shape == 3 || shape == 4; }

// The compiled shape that runs a policy with two hidden layers: the narrowest one whose hidden
// widths cover the policy's (the kernels pad narrower layers with zeros); -1 if none does.
int rollout_mlp_tiled_shape(uint32_t task, uint32_t n_layers, const uint32_t* sizes)
{
    if (n_layers != 3) return -1;
    int best = -1;
    for (int i = 0; i < static_cast<int>(sizeof(kShapes) / sizeof(kShapes[0])); ++i) {
        const TiledShape& s = kShapes[i];
        if (s.task == task && s.nin == sizes[0] && s.nout == sizes[3] && s.h1 >= sizes[1] && s.h2 >= sizes[2] &&
            (best < 0 || s.h1 < kShapes[best].h1))
            best = i;
    }
    return best;
}

// episodes per block; the wider cart-pole shapes switch to the warp-specialised kernel
// (two groups of 8) once a member has more than 8 episodes
uint32_t rollout_mlp_tiled_eb(int shape, uint32_t episodes)
{
    if (has_two_group_kernel(shape) && episodes > kShapes[shape].EB) return 2u * kShapes[shape].EB;
    return kShapes[shape].EB;
}

template <class K>
static int launch_one(K kernel, int threads, size_t act_floats, cudaStream_t st, const RolloutMlpArgs& a,
                      DeviceStatus* status)
{
    const size_t bytes = (static_cast<size_t>(a.ldD) + act_floats) * sizeof(float);
    if (bytes > 220u * 1024u) return -2;
    if (!a.attr_done &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess)
        return -1;
    dim3 grid(a.P, a.n_eb);
    return launch_dependent(kernel, grid, dim3(threads), bytes, st, a, status) == cudaSuccess ? 1 : -1;
}

int launch_rollout_mlp_tiled(cudaStream_t st, const RolloutMlpArgs& a, DeviceStatus* status)
{
    const int shape = rollout_mlp_tiled_shape(a.task, a.n_layers, a.sizes);
    if (shape < 0) return -2;
    if (has_two_group_kernel(shape) && a.EB == 2u * kShapes[shape].EB) {
        if (shape == 1)
            return launch_one(k_rollout_cartpole_ws<64, 64, 8, 64, 2, 1, 1, 4, 4, 1, 32>, 32 + 64 * 2,
                              (2 * 5 + 64 + 2 * 64) * 8, st, a, status);
        if (shape == 3)
            return launch_one(k_rollout_cartpole_ws<32, 32, 8, 32, 2, 1, 1, 4, 4, 1, 32>, 32 + 32 * 2,
                              (2 * 5 + 32 + 2 * 32) * 8, st, a, status);
        return launch_one(k_rollout_cartpole_ws<128, 128, 8, 128, 2, 1, 1, 4, 4, 1, 32>, 32 + 128 * 2,
                          (2 * 5 + 128 + 2 * 128) * 8, st, a, status);
    }
    if (a.EB != kShapes[shape].EB) return -2;
    switch (shape) {
        case 0:
            return launch_one(k_rollout_mlp_tiled<5, 16, 16, 1, 1, 32, EVO_TASK_CARTPOLE, 1, 1, 1, 2, 1, 16>,
                              32, (2 * 5 + 16 + 16 + 1) * 1, st, a, status);
        case 1:
            return launch_one(k_rollout_mlp_tiled<5, 64, 64, 1, 8, 64, EVO_TASK_CARTPOLE, 1, 1, 4, 4, 1, 32>,
                              64, (2 * 5 + 64 + 64 + 1) * 8, st, a, status);
        case 2:
            return launch_one(k_rollout_mlp_tiled<28, 128, 128, 8, 4, 128, EVO_TASK_TANH_LINEAR, 4, 4, 8, 8, 1, 16>,
                              128, (2 * 36 + 128 + 128 + 8) * 4, st, a, status);
        case 3:
            return launch_one(k_rollout_mlp_tiled<5, 32, 32, 1, 8, 32, EVO_TASK_CARTPOLE, 1, 1, 4, 4, 1, 32>,
                              32, (2 * 5 + 32 + 32 + 1) * 8, st, a, status);
        case 4:
            return launch_one(k_rollout_mlp_tiled<5, 128, 128, 1, 8, 128, EVO_TASK_CARTPOLE, 1, 1, 4, 4, 1, 32>,
                              128, (2 * 5 + 128 + 128 + 1) * 8, st, a, status);
    }
    return -2;
}

}  // namespace evo
