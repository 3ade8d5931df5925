// Large-population control roll-out (tanh-linear task, MLP 28-128-128-8) on the tensor cores.
//
// A member's two wide layers are the A operands of tcgen05.mma and stay on chip for all T steps:
// W (128 x K) as two fp16 parts, w = hi + lo with hi = fp16(w) and lo = fp16(w - hi) (22 mantissa
// bits together; every product of two fp16 numbers is exact and sums accumulate in fp32, so the
// layer is as accurate as an fp32 FMA chain; weights beyond +-65,504, the fp16 range, are clamped to
// it).  The hi part of W2 and both parts of W1 live in
// tensor memory, the lo part of W2 in shared memory.  The B operand of a layer is the activation
// block of the member's four episodes, also as two fp16 parts set side by side, N = 8 columns
// [hi(e0..e3) | lo(e0..e3)]: one MMA with A = W_part then yields W_part . a_hi and W_part . a_lo at once
// and the epilogue adds the two column groups, so all four cross terms are kept and a layer costs
// two MMAs per 16 inputs.
//
// One block per SM runs four TEAMS of 128 threads; a team owns one (member, episode block) at a
// time, 128 columns of tensor memory and its own mbarrier.  Thread r of a team is row r of the
// hidden layers (tensor-memory lane r).  Every warp of a team issues its own share of a layer's
// MMAs (one elected lane each: a single thread can only start an MMA every ~50 clocks) into its own
// 8-column accumulator and commits to the team's mbarrier; the epilogue reads the four
// accumulators, adds bias, applies tanh, splits into fp16 parts and writes the next B operand with
// one 16-byte store per thread.  The narrow layers (action 128 -> 8, task dynamics 36 -> 28) run on
// the fp32 pipe with the hidden layer in fp32.  While one team waits for its MMAs or sits in an
// epilogue the other three use the SM: the per-step chain of a member (two MMA batches, four
// tanh layers) is latency, and four members per SM overlap it.
//
// Paper: Section 2 (roll-out loop, central seeds), Section 4 (get_actions over the population with
// parameters as data; stateless task step; identical initial observations for all members).
#include "internal.h"
#include "umma.cuh"
#include "noise.cuh"
#include "fp32x2.cuh"

#include <cuda_fp16.h>

namespace evo {
namespace tl {

constexpr int kH = 128;                 // hidden width = MMA M
constexpr int kNx = 28, kNa = 8;        // task state and action widths
constexpr int kK1 = 32;                 // layer-1 inputs padded to two K steps of 16
constexpr int kEB = 4;                  // episodes per team item
constexpr int kTeams = 4, kTeamThreads = 128, kThreads = kTeams * kTeamThreads;
// tensor-memory columns of a team
constexpr uint32_t kColW2hi = 0, kColW1hi = 64, kColW1lo = 80, kColAcc = 96, kColsTeam = 128;
// clocks the layer-2 MMA batch of one team keeps the tensor pipe busy (16 MMAs of ~25 clocks); measured
// optimum of the spacing between two teams' batches (200..600 all help, 450 is best, 1000 throttles;
// spacing the short layer-1 batches as well costs more than it gains)
constexpr unsigned long long kL2Gap = 450;
constexpr int kH2Pitch = kH + 32;       // h2 rows in shared memory, 4 floats of skew per 16
constexpr int kB1Lbo = 144;             // layer-1 B operand: bytes between its 8-input groups (skewed: no bank conflicts)

struct TeamSmem {
    alignas(128) unsigned char w2lo[kH * kH * 2];    // fp16, K-major 8x8 core matrices (A operand)
    alignas(128) unsigned char b1[640];              // layer-1 B operand, K-major: (k, n) at (k/8) 144 + 16 n + 2 (k%8)
    alignas(128) unsigned char b2[kH * 16];          // layer-2 B operand, N-major: [k][hi e0..3 | lo e0..3] fp16
    alignas(16) float h2[kEB][kH2Pitch];             // second hidden layer, fp32, [episode][unit]
    alignas(16) float x[kEB][32];                    // task state, fp32
    alignas(16) float act[kEB][kNa];                 // action, fp32
    alignas(8) uint64_t bar;                         // MMA batches of this team
    float ret[kEB];
    int abort;
};
struct Smem {
    TeamSmem team[kTeams];
    alignas(16) float dyn[kNx][36];                  // [A | B] of the task, row i = output i
    alignas(8) uint64_t drain_bar;
    unsigned long long next_l2_slot;                 // clock at which the next team may start its layer-2 batch
    uint32_t tmem_slot;
};

__host__ __device__ constexpr uint32_t idesc_f16(uint32_t M, uint32_t N, bool b_mn_major)
{
    // c = f32, a = b = f16, A K-major (or tensor memory), B as given
    return (1u << 4) | (b_mn_major ? (1u << 16) : 0u) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* u)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Pre-activations of this thread's row from the team's four accumulators (8 columns each: the
// products with the hi parts of the four episodes' activations, then those with the lo parts):
// pre[e] = bias + sum over the accumulators of (col e + col 4+e).  Two 16-column loads, so that only
// 16 registers are live at a time.
__device__ __forceinline__ void acc_sums(uint32_t taddr, float bias, float* pre)
{
    float v[16];
    tmem_ld16(taddr, v);
#pragma unroll
    for (int e = 0; e < 4; ++e) pre[e] = bias + ((v[e] + v[4 + e]) + (v[8 + e] + v[12 + e]));
    tmem_ld16(taddr + 16u, v);
#pragma unroll
    for (int e = 0; e < 4; ++e) pre[e] += (v[e] + v[4 + e]) + (v[8 + e] + v[12 + e]);
}

// tanh(x) = 1 - 2/(exp(2x)+1) on the special-function unit; absolute error ~2e-7
__device__ __forceinline__ float tanh_sfu(float x)
{
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 2.885390082f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.0f));
    return fmaf(-2.0f, r, 1.0f);
}

// x = hi + lo with both parts fp16 (round to nearest)
__device__ __forceinline__ void split_f16(float x, __half& hi, __half& lo)
{
    hi = __float2half_rn(x);
    lo = __float2half_rn(x - __half2float(hi));
}
// weights of the wide layers: magnitudes above the largest fp16 number are taken as that number (the
// tanh behind them is saturated long before; without the clamp they would turn into infinities)
__device__ __forceinline__ void split_weight(float w, __half& hi, __half& lo)
{
    split_f16(fminf(fmaxf(w, -65504.0f), 65504.0f), hi, lo);
}
__device__ __forceinline__ uint32_t pack_h2(__half a, __half b)      // a in the low half
{
    return static_cast<uint32_t>(__half_as_ushort(a)) | (static_cast<uint32_t>(__half_as_ushort(b)) << 16);
}

// The teams share the tensor pipe and run the same chain with the same period.  Left alone, their
// MMA batches interleave in the pipe (two batches issued together both finish late) and the teams
// bunch up.  A team therefore books the pipe before it issues a batch: slots are handed out in
// order of arrival, `clocks` apart (about the time the batch keeps the pipe busy), and a team that
// is early sleeps until its slot (bounded: the loop ends after 64 short sleeps in any case).
__device__ __forceinline__ void book_tensor_pipe(unsigned long long* next_slot, unsigned long long clocks)
{
    if (clocks == 0ull) return;
    const unsigned long long now = static_cast<unsigned long long>(clock64());
    unsigned long long old = *reinterpret_cast<volatile unsigned long long*>(next_slot), mine;
    for (;;) {
        mine = old > now ? old : now;
        const unsigned long long seen = atomicCAS(next_slot, old, mine + clocks);
        if (seen == old) break;
        old = seen;
    }
    for (int i = 0; i < 64 && static_cast<unsigned long long>(clock64()) < mine; ++i) __nanosleep(40);
}

__device__ __forceinline__ void team_sync(int team)
{
    asm volatile("bar.sync %0, %1;" :: "r"(1 + team), "n"(kTeamThreads) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
k_rollout_tl_tc(const RolloutMlpArgs a, DeviceStatus* status)
{
    dep_wait();
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem& S = *reinterpret_cast<Smem*>(smem_raw);
    const int tid = threadIdx.x;
    const int team = tid / kTeamThreads, r = tid % kTeamThreads;     // r = hidden unit = tensor-memory lane
    const int w = r / 32, l = r % 32;                                // team-local warp and lane
    TeamSmem& T = S.team[team];
    const PhiloxKey key = philox_key(a.k0, a.k1);

    // ---- block set-up: task matrices, barriers, tensor memory ---------------------------------------
    for (int i = tid; i < kNx * 36; i += kThreads) {
        const int row = i / 36, col = i % 36;
        S.dyn[row][col] = col < kNx ? a.task_const[row * kNx + col] : a.task_const[kNx * kNx + row * kNa + (col - kNx)];
    }
    for (int i = r; i < 640 / 4; i += kTeamThreads) reinterpret_cast<uint32_t*>(T.b1)[i] = 0u;   // inputs 28..31 stay zero
    if (r == 0) { mbar_init(smem_u32(&T.bar), 4); mbar_init_fence(); T.abort = 0; }
    if (tid == 0) { mbar_init(smem_u32(&S.drain_bar), kTeams * 4); mbar_init_fence(); S.next_l2_slot = 0ull; }
    if (tid < 32) tmem_alloc(smem_u32(&S.tmem_slot), 512);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = S.tmem_slot + static_cast<uint32_t>(team) * kColsTeam;   // the team's columns
    const uint32_t tm_lane = tm + (static_cast<uint32_t>(w * 32) << 16);          // this warp's lanes
    const uint32_t bar = smem_u32(&T.bar);
    uint32_t parity = 0;

    // operand descriptors of this warp's MMAs (only lane 0 issues)
    constexpr uint32_t kIdescL1 = idesc_f16(kH, 8, false), kIdescL2 = idesc_f16(kH, 8, true);
    //   layer 1: warp w takes part (w & 1) of W1 and K step (w >> 1)
    const uint32_t l1_a = tm + ((w & 1) ? kColW1lo : kColW1hi) + 8u * static_cast<uint32_t>(w >> 1);
    const uint64_t l1_b = umma_smem_desc(smem_u32(T.b1) + static_cast<uint32_t>(w >> 1) * 2u * kB1Lbo, kB1Lbo, 128u);
    //   layer 2: warp w takes K steps 2w and 2w+1, both parts of W2 (the second step's operands lie 256
    //   bytes = 16 descriptor units further on)
    const uint32_t l2_a0 = tm + kColW2hi + 8u * static_cast<uint32_t>(2 * w);
    const uint64_t l2_b0 = umma_smem_desc(smem_u32(T.b2) + static_cast<uint32_t>(2 * w) * 256u, 128u, 128u);
    const uint64_t l2_s0 = umma_smem_desc(smem_u32(T.w2lo) + static_cast<uint32_t>(2 * w) * 256u, 128u, 2048u);
    const uint32_t acc_w = tm + kColAcc + 8u * static_cast<uint32_t>(w);
    const bool drop_first_commit = (status->debug_flags & EVO_DEBUG_DROP_COMPLETION) != 0u;

    // the narrow layers use another thread mapping: warp = episode; for the action layer lane = (eighth
    // q8 of the 128 inputs, pair op of the 8 outputs), for the task dynamics lane = output i
    const int e = w, q8 = l & 7, op = l >> 3, di = min(l, kNx - 1);
    float dynw[36];                                   // row di of [A | B]
#pragma unroll
    for (int j = 0; j < 36; ++j) dynw[j] = S.dyn[di][j];
    const bool tracing = a.trace != nullptr;
    volatile int* const aborted = &T.abort;

    // the four teams run the same chain with the same period: started together they would all want
    // the tensor pipe at the same moment and then all leave it idle, so team t starts t/4 step late
    if (team > 0) __nanosleep(static_cast<uint32_t>(team) * 500u);
    const uint32_t items = a.P * a.n_eb;
    // items go to the blocks round-robin first and to a block's teams second, so that a small
    // population spreads over all SMs before any SM runs two members at a time
    for (uint32_t item = blockIdx.x + gridDim.x * team; item < items; item += gridDim.x * kTeams) {
        const uint32_t member = item / a.n_eb, eb = item % a.n_eb;
        const uint32_t e0 = eb * kEB;
        const bool full_width = a.sizes[1] == kH && a.sizes[2] == kH;
        const int nE = min(static_cast<uint32_t>(kEB), a.E - e0);
        const float* th = a.theta + static_cast<size_t>(member) * a.ldD;
        // offsets in the flat parameter row; hidden widths h1, h2 <= 128 (narrower layers are padded with
        // zero rows and columns, so the padded units are tanh(0) = 0 and feed nothing onwards)
        const int h1 = static_cast<int>(a.sizes[1]), h2 = static_cast<int>(a.sizes[2]);
        const int kOffW1 = 0, kOffB1 = h1 * kNx, kOffW2 = kOffB1 + h1, kOffB2 = kOffW2 + h2 * h1,
                  kOffW3 = kOffB2 + h2, kOffB3 = kOffW3 + kNa * h2;

        // ---- the member's weights: registers -> tensor memory / shared memory ---------------------
        {   // W1 row r (28 inputs, padded with zeros to 32): both parts into tensor memory
            float wrow[kK1];
#pragma unroll
            for (int c = 0; c < kNx / 4; ++c) {             // rows are 112 bytes: 16-byte aligned
                const float4 v = r < h1 ? __ldg(reinterpret_cast<const float4*>(th + kOffW1 + r * kNx) + c)
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                wrow[4 * c] = v.x; wrow[4 * c + 1] = v.y; wrow[4 * c + 2] = v.z; wrow[4 * c + 3] = v.w;
            }
#pragma unroll
            for (int k = kNx; k < kK1; ++k) wrow[k] = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    __half ha, la, hb, lb;
                    split_weight(wrow[16 * c + 2 * i], ha, la);
                    split_weight(wrow[16 * c + 2 * i + 1], hb, lb);
                    hi[i] = pack_h2(ha, hb); lo[i] = pack_h2(la, lb);
                }
                tmem_st8(tm_lane + kColW1hi + 8u * c, hi);
                tmem_st8(tm_lane + kColW1lo + 8u * c, lo);
            }
        }
#pragma unroll 1
        for (int c = 0; c < kH / 16; ++c) {   // W2 row r, 16 inputs at a time: hi -> tensor memory, lo -> shared memory
            float wv[16];
            if (full_width) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(th + kOffW2 + r * kH + 16 * c) + j);
                    wv[4 * j] = v.x; wv[4 * j + 1] = v.y; wv[4 * j + 2] = v.z; wv[4 * j + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    wv[j] = (r < h2 && 16 * c + j < h1) ? __ldg(th + kOffW2 + r * h1 + 16 * c + j) : 0.f;
            }
            uint32_t hi[8], lo[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                __half ha, la, hb, lb;
                split_weight(wv[2 * i], ha, la);
                split_weight(wv[2 * i + 1], hb, lb);
                hi[i] = pack_h2(ha, hb); lo[i] = pack_h2(la, lb);
            }
            tmem_st8(tm_lane + kColW2hi + 8u * c, hi);
            // core matrix (row group r/8, K chunk): 8 rows x 16 bytes; K chunks 128 B apart, row groups 2048 B
            unsigned char* dst = T.w2lo + (r >> 3) * 2048 + (2 * c) * 128 + (r & 7) * 16;
            *reinterpret_cast<uint4*>(dst) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            *reinterpret_cast<uint4*>(dst + 128) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
        tmem_st_wait();
        const float bias1 = r < h1 ? __ldg(th + kOffB1 + r) : 0.f, bias2 = r < h2 ? __ldg(th + kOffB2 + r) : 0.f;
        float w3[2][16];                        // action layer: rows 2 op and 2 op + 1, inputs 16 q8 .. 16 q8 + 15
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 16; ++j)
                w3[i][j] = (16 * q8 + j < h2) ? __ldg(th + kOffW3 + (2 * op + i) * h2 + 16 * q8 + j) : 0.f;
        const float bias3a = __ldg(th + kOffB3 + 2 * op), bias3b = __ldg(th + kOffB3 + 2 * op + 1);

        // ---- reset: seeded start states, the same for every member ----------------------------------
        if (r < kEB * (kNx / 4)) {
            const int ee = r / (kNx / 4), qq = r % (kNx / 4);
            const float4 z = stream_normal4(key, 1u, status->generation, e0 + min(ee, nE - 1), qq);
            const float zs[4] = { z.x, z.y, z.z, z.w };
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                __half hi, lo;
                split_f16(zs[j], hi, lo);
                const int k = 4 * qq + j;
                T.x[ee][k] = zs[j];
                unsigned char* bp = T.b1 + (k >> 3) * kB1Lbo + (k & 7) * 2;
                *reinterpret_cast<__half*>(bp + ee * 16) = hi;
                *reinterpret_cast<__half*>(bp + (4 + ee) * 16) = lo;
            }
        }
        fence_async_smem();
        tc_fence_before();
        team_sync(team);
        float xcur = T.x[e][di];                // this thread's state component (lanes 28..31 mirror 27)
        float ret = 0.f;

        // ---- time loop ----------------------------------------------------------------------------------
        for (uint32_t t = 0; t < a.T; ++t) {
            // layer 1: one MMA per warp
            if (l == 0 && !*aborted) {
                tc_fence_after();
                mma_f16_ts(acc_w, l1_a, l1_b, kIdescL1, 0u);
                if (!(drop_first_commit && t == 0u)) umma_commit(bar);
            }
            __syncwarp();
            wait_or_abort(&T.abort, &T.bar, parity, status); parity ^= 1u;
            tc_fence_after();
            {
                float pre[kEB];
                acc_sums(tm_lane + kColAcc, bias1, pre);
                uint32_t pk[4];
                __half hh[kEB], hl[kEB];
#pragma unroll
                for (int ee = 0; ee < kEB; ++ee) split_f16(tanh_sfu(pre[ee]), hh[ee], hl[ee]);
                pk[0] = pack_h2(hh[0], hh[1]); pk[1] = pack_h2(hh[2], hh[3]);
                pk[2] = pack_h2(hl[0], hl[1]); pk[3] = pack_h2(hl[2], hl[3]);
                *reinterpret_cast<uint4*>(T.b2 + r * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            fence_async_smem();
            tc_fence_before();
            if (r == 0) book_tensor_pipe(&S.next_l2_slot, kL2Gap);
            team_sync(team);
            // layer 2: four MMAs per warp (two K steps x two parts of W2)
            if (l == 0 && !*aborted) {
                tc_fence_after();
                // (umma_bf16 is the kind::f16 MMA with A from shared memory; the operand type, fp16 here,
                // comes from the instruction descriptor)
                mma_f16_ts(acc_w, l2_a0, l2_b0, kIdescL2, 0u);
                umma_bf16(acc_w, l2_s0, l2_b0, kIdescL2, 1u);
                mma_f16_ts(acc_w, l2_a0 + 8u, l2_b0 + 16u, kIdescL2, 1u);
                umma_bf16(acc_w, l2_s0 + 16u, l2_b0 + 16u, kIdescL2, 1u);
                umma_commit(bar);
            }
            __syncwarp();
            wait_or_abort(&T.abort, &T.bar, parity, status); parity ^= 1u;
            tc_fence_after();
            {
                float pre[kEB];
                acc_sums(tm_lane + kColAcc, bias2, pre);
                const int rs = r + (r >> 4) * 4;               // skewed column
#pragma unroll
                for (int ee = 0; ee < kEB; ++ee) T.h2[ee][rs] = tanh_sfu(pre[ee]);
            }
            tc_fence_before();
            team_sync(team);
            // action layer on the fp32 pipe: warp = episode e, lane = (input eighth q8, output pair op)
            {
                const float4* hp = reinterpret_cast<const float4*>(&T.h2[e][20 * q8]);
                // two inputs per paired FMA (fma.rn.f32x2): half the instructions of the scalar form
                float2 s01 = make_float2(0.f, 0.f), s23 = s01, u01 = s01, u23 = s01;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 hv = hp[j];
                    const float2 h01 = make_float2(hv.x, hv.y), h23 = make_float2(hv.z, hv.w);
                    ffma2(s01, make_float2(w3[0][4 * j], w3[0][4 * j + 1]), h01);
                    ffma2(u01, make_float2(w3[1][4 * j], w3[1][4 * j + 1]), h01);
                    ffma2(s23, make_float2(w3[0][4 * j + 2], w3[0][4 * j + 3]), h23);
                    ffma2(u23, make_float2(w3[1][4 * j + 2], w3[1][4 * j + 3]), h23);
                }
                float sa = (s01.x + s01.y) + (s23.x + s23.y), sb = (u01.x + u01.y) + (u23.x + u23.y);
#pragma unroll
                for (int off = 1; off < 8; off <<= 1) {
                    sa += __shfl_xor_sync(0xffffffffu, sa, off);
                    sb += __shfl_xor_sync(0xffffffffu, sb, off);
                }
                const float aa = a.action_scale * tanh_sfu(sa + bias3a), ab = a.action_scale * tanh_sfu(sb + bias3b);
                if (q8 == 0) {
                    *reinterpret_cast<float2*>(&T.act[e][2 * op]) = make_float2(aa, ab);
                    ret = fmaf(-0.01f * aa, aa, ret);
                    ret = fmaf(-0.01f * ab, ab, ret);
                }
            }
            __syncwarp();
            // task dynamics x' = tanh(A x + B a): warp = episode e, lane = output i
            {
                if (l < kNx) ret = fmaf(-xcur, xcur, ret);        // reward on (x_t, a_t)
                const float4* xp = reinterpret_cast<const float4*>(&T.x[e][0]);
                const float4* ap = reinterpret_cast<const float4*>(&T.act[e][0]);
                float2 s01 = make_float2(0.f, 0.f), s23 = s01;
#pragma unroll
                for (int j = 0; j < kNx / 4; ++j) {
                    const float4 xv = xp[j];
                    ffma2(s01, make_float2(dynw[4 * j], dynw[4 * j + 1]), make_float2(xv.x, xv.y));
                    ffma2(s23, make_float2(dynw[4 * j + 2], dynw[4 * j + 3]), make_float2(xv.z, xv.w));
                }
#pragma unroll
                for (int j = 0; j < kNa / 4; ++j) {
                    const float4 av = ap[j];
                    ffma2(s01, make_float2(dynw[kNx + 4 * j], dynw[kNx + 4 * j + 1]), make_float2(av.x, av.y));
                    ffma2(s23, make_float2(dynw[kNx + 4 * j + 2], dynw[kNx + 4 * j + 3]), make_float2(av.z, av.w));
                }
                const float xn = tanh_sfu((s01.x + s01.y) + (s23.x + s23.y));
                __syncwarp();                                      // every lane has read x[e][.]
                if (l < kNx) {
                    __half hi, lo;
                    split_f16(xn, hi, lo);
                    T.x[e][l] = xn;
                    unsigned char* bp = T.b1 + (l >> 3) * kB1Lbo + (l & 7) * 2;
                    *reinterpret_cast<__half*>(bp + e * 16) = hi;
                    *reinterpret_cast<__half*>(bp + (4 + e) * 16) = lo;
                    if (tracing && t < a.trace_T && e < nE &&
                        EVO_IN_BOUNDS(status, EVO_SITE_TRACE, ((static_cast<size_t>(member) * a.E + e0 + e) * a.trace_T + t) * kNx + l,
                                      static_cast<size_t>(a.P) * a.E * a.trace_T * kNx))
                        a.trace[((static_cast<size_t>(member) * a.E + e0 + e) * a.trace_T + t) * kNx + l] = xn;
                }
                xcur = xn;
            }
            fence_async_smem();
            tc_fence_before();
            team_sync(team);
        }

        // ---- the item's return: episodes summed in order (fixed tree inside a warp) ------------------
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ret += __shfl_xor_sync(0xffffffffu, ret, off);
        if (l == 0) T.ret[e] = ret;
        team_sync(team);
        if (r == 0) {
            float v = 0.f;
            for (int ee = 0; ee < nE; ++ee) v += T.ret[ee];
            // after a time-out the numbers mean nothing: report NaN, which makes tell skip the update
            if (EVO_IN_BOUNDS(status, EVO_SITE_FIT_PARTIAL, static_cast<size_t>(member) * a.n_eb + eb,
                              static_cast<size_t>(a.P) * a.n_eb))
                a.fit_partial[static_cast<size_t>(member) * a.n_eb + eb] = T.abort ? __int_as_float(0x7FC00000) : v;
        }
        team_sync(team);
    }

    // ---- leave: after a time-out MMAs may still be running (a commit covers the MMAs its own thread
    // issued, so every issuing thread commits once more); the block gives them one bounded wait
    __syncthreads();
    bool any_abort = false;
#pragma unroll
    for (int i = 0; i < kTeams; ++i) any_abort |= S.team[i].abort != 0;
    if (any_abort) {
        if (l == 0) umma_commit(smem_u32(&S.drain_bar));
        if (tid == 0) mbar_wait_bounded(smem_u32(&S.drain_bar), 0u, &status->wait_cycles_log2);
        __syncthreads();
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32) tmem_dealloc(S.tmem_slot, 512);
}

}  // namespace tl

bool rollout_tl_tc_supported(const RolloutMlpArgs& a)
{
    return a.task == EVO_TASK_TANH_LINEAR && a.n_layers == 3 && a.sizes[0] == tl::kNx && a.sizes[1] <= tl::kH &&
           a.sizes[2] <= tl::kH && a.sizes[3] == tl::kNa && a.EB == tl::kEB;
}

int launch_rollout_tl_tc(cudaStream_t st, const RolloutMlpArgs& a, DeviceStatus* status)
{
    if (!rollout_tl_tc_supported(a)) return -2;
    const size_t bytes = sizeof(tl::Smem);
    if (!a.attr_done &&
        cudaFuncSetAttribute(tl::k_rollout_tl_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess)
        return -1;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    const uint32_t items = a.P * a.n_eb;
    const uint32_t blocks = min(static_cast<uint32_t>(sms), items);
    launch_dependent(tl::k_rollout_tl_tc, dim3(blocks), dim3(tl::kThreads), bytes, st, a, status);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace evo
