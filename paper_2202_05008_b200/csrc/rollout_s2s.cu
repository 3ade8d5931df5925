// Sequence-to-sequence addition task with an LSTM encoder-decoder policy (paper Section 3,
// "Seq2Seq Learning"): a single-step task whose fitness is minus the mean cross-entropy of the
// answer digits over a batch of queries that every member sees.
//
// Conventions: tokens '0'..'9' -> 0..9, '+' -> 10, '=' -> 11; the encoder reads "a+b" (2 nd + 1
// tokens), the decoder is fed '=' and then the true answer digits and must produce the nd + 1
// digits of the sum; gate order (input, forget, cell, output); flat parameters enc.Wx[4h][12],
// enc.Wh[4h][h], enc.b[4h], dec.*, out.W[12][h], out.b[12].  A cell's pre-activation is one
// contraction [Wh | Wx | b] . [h; onehot(token); 1] with bf16 operands and fp32 accumulation; the
// read-out out.W . h likewise.
//
//   k_s2s_simple  CUDA cores, one block per (member, 16 queries): the plain version.
//   k_s2s_tc      tcgen05, one block per (member, 128 queries), one block per SM.  The member's
//                 [4h = 512] x [K = 144] weight tile (bf16, 144 KB) stays in shared memory for a
//                 whole phase (encoder, then decoder); the B operand is the hidden state of the 128
//                 queries plus their one-hot token and a constant 1, so one chain of 9 MMAs per gate
//                 produces the complete pre-activation in TMEM (2 halves x 4 gates x 64 columns =
//                 all 512 columns).  The queries are two halves of 64 whose steps alternate: while
//                 the epilogue warps of one half apply the gate non-linearities (thread = hidden
//                 unit = TMEM lane, cell state in registers) and write the new hidden state straight
//                 back into the B operand, the tensor cores work on the other half.  The rows of the
//                 sigmoid gates are halved when staged, so every non-linearity is one tanh of the
//                 special-function unit; that unit (5 tanh per cell and step) is what bounds the
//                 kernel, not the tensor cores.  The decoder's read-out runs on the CUDA cores from
//                 the B operand while the next step's MMAs are in flight; its logits are kept and
//                 the cross-entropy is taken once per item.  The next cell's weights are prefetched
//                 into L2 while the current phase computes.  Every wait is bounded.
#include "internal.h"
#include "async.cuh"
#include "noise.cuh"
#include "umma.cuh"
#include "fp32x2.cuh"

namespace evo {

constexpr int kVocab = 12;
constexpr int kTokPlus = 10, kTokEq = 11;
constexpr int kS2sMaxDigits = 4;
constexpr int kS2sMaxTe = 2 * kS2sMaxDigits + 1, kS2sMaxTd = kS2sMaxDigits + 1;

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Query i of a generation: a, b uniform on [0, 10^nd) from the first two words of stream 6.
__device__ __forceinline__ void s2s_query(const PhiloxKey& key, uint32_t generation, uint32_t i, uint32_t nd,
                                          uint8_t* enc, uint8_t* dec, uint8_t* tgt)
{
    uint32_t range = 1;
    for (uint32_t k = 0; k < nd; ++k) range *= 10u;
    const uint4 w = philox4x32_10(i, 0u, generation, 6u, key);
    const uint32_t a = __umulhi(w.x, range), b = __umulhi(w.y, range), sum = a + b;
    uint32_t div = range / 10u;
    for (uint32_t k = 0; k < nd; ++k, div /= 10u) {
        enc[k] = static_cast<uint8_t>((a / div) % 10u);
        enc[nd + 1 + k] = static_cast<uint8_t>((b / div) % 10u);
    }
    enc[nd] = kTokPlus;
    div = range;
    for (uint32_t k = 0; k <= nd; ++k, div /= 10u) tgt[k] = static_cast<uint8_t>((sum / div) % 10u);
    dec[0] = kTokEq;
    for (uint32_t k = 1; k <= nd; ++k) dec[k] = tgt[k - 1];
}

__device__ __forceinline__ float sigmoid_acc(float x) { return 1.0f / (1.0f + expf(-x)); }

// cross-entropy of one position from its 12 logits
__device__ __forceinline__ float token_loss(const float* lg, int target)
{
    float mx = lg[0];
#pragma unroll
    for (int o = 1; o < kVocab; ++o) mx = fmaxf(mx, lg[o]);
    float se = 0.f;
#pragma unroll
    for (int o = 0; o < kVocab; ++o) se += expf(lg[o] - mx);
    return (mx + logf(se)) - lg[target];
}

struct S2sArgs {
    const float* theta; uint32_t ldD, P;
    uint32_t h, nd, B;
    uint32_t k0, k1;
    const DeviceStatus* status;  // holds the generation counter
    float* partial;              // [P][n_chunks] sums of token losses
    uint32_t n_chunks;
    float* logits;               // nullable: [P][B][nd+1][12] (simple kernel only)
};

// ------------------------------------------------------------------------------------------
// CUDA-core version: thread = hidden unit, 16 queries per block, weights read through the caches.
// ------------------------------------------------------------------------------------------
constexpr int kSimpleQ = 16;

__global__ void __launch_bounds__(128)
k_s2s_simple(const S2sArgs a)
{
    __shared__ __align__(16) float hs[kSimpleQ][128];           // bf16-rounded hidden state
    __shared__ float lg[kSimpleQ][kVocab];
    __shared__ uint8_t enc[kSimpleQ][kS2sMaxTe], dec[kSimpleQ][kS2sMaxTd], tgt[kSimpleQ][kS2sMaxTd];
    __shared__ float loss_s[kSimpleQ];
    const uint32_t h = a.h, r = threadIdx.x, member = blockIdx.x, q0 = blockIdx.y * kSimpleQ;
    const uint32_t nq = min(static_cast<uint32_t>(kSimpleQ), a.B - q0);
    const uint32_t Te = 2 * a.nd + 1, Td = a.nd + 1;
    const PhiloxKey key = philox_key(a.k0, a.k1);
    if (r < kSimpleQ) {
        s2s_query(key, a.status->generation, q0 + min(r, nq - 1u), a.nd, enc[r], dec[r], tgt[r]);
        loss_s[r] = 0.f;
    }
    for (uint32_t s = 0; s < kSimpleQ; ++s) hs[s][r] = 0.f;
    float c[kSimpleQ];
#pragma unroll
    for (int s = 0; s < kSimpleQ; ++s) c[s] = 0.f;
    const float* p = a.theta + static_cast<size_t>(member) * a.ldD;
    const size_t cell = static_cast<size_t>(4) * h * kVocab + static_cast<size_t>(4) * h * h + 4u * h;
    const float* oW = p + 2 * cell;
    const float* ob = oW + static_cast<size_t>(kVocab) * h;
    __syncthreads();

    for (uint32_t t = 0; t < Te + Td; ++t) {
        const bool decoding = t >= Te;
        const float* Wx = p + (decoding ? cell : 0);
        const float* Wh = Wx + static_cast<size_t>(4) * h * kVocab;
        const float* bb = Wh + static_cast<size_t>(4) * h * h;
        float acc[4][kSimpleQ];
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int s = 0; s < kSimpleQ; ++s) acc[g][s] = 0.f;
        if (r < h) {
            for (uint32_t k = 0; k < h; k += 4) {
                float4 w[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    w[g] = __ldg(reinterpret_cast<const float4*>(Wh + (static_cast<size_t>(g) * h + r) * h + k));
                    w[g].x = bf16_round(w[g].x); w[g].y = bf16_round(w[g].y);
                    w[g].z = bf16_round(w[g].z); w[g].w = bf16_round(w[g].w);
                }
#pragma unroll
                for (int s = 0; s < kSimpleQ; ++s) {
                    const float4 x = *reinterpret_cast<const float4*>(&hs[s][k]);
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        acc[g][s] = fmaf(w[g].x, x.x, acc[g][s]);
                        acc[g][s] = fmaf(w[g].y, x.y, acc[g][s]);
                        acc[g][s] = fmaf(w[g].z, x.z, acc[g][s]);
                        acc[g][s] = fmaf(w[g].w, x.w, acc[g][s]);
                    }
                }
            }
        }
        __syncthreads();                                       // every thread is done reading hs
        if (r < h) {
            float bias[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) bias[g] = bf16_round(bb[g * h + r]);
#pragma unroll
            for (int s = 0; s < kSimpleQ; ++s) {
                const uint32_t tok = decoding ? dec[s][t - Te] : enc[s][t];
                float pre[4];
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    pre[g] = acc[g][s] + bf16_round(Wx[(static_cast<size_t>(g) * h + r) * kVocab + tok]) + bias[g];
                const float ig = sigmoid_acc(pre[0]), fg = sigmoid_acc(pre[1]);
                const float gg = tanhf(pre[2]), og = sigmoid_acc(pre[3]);
                c[s] = fmaf(fg, c[s], ig * gg);
                hs[s][r] = bf16_round(og * tanhf(c[s]));
            }
        }
        __syncthreads();
        if (decoding) {
            for (uint32_t idx = r; idx < kSimpleQ * kVocab; idx += blockDim.x) {
                const uint32_t s = idx / kVocab, o = idx % kVocab;
                float v = 0.f;
                for (uint32_t k = 0; k < h; ++k) v = fmaf(bf16_round(oW[o * h + k]), hs[s][k], v);
                lg[s][o] = v + ob[o];
                if (a.logits && s < nq)
                    a.logits[((static_cast<size_t>(member) * a.B + q0 + s) * Td + (t - Te)) * kVocab + o] = lg[s][o];
            }
            __syncthreads();
            if (r < nq) loss_s[r] += token_loss(lg[r], tgt[r][t - Te]);
            __syncthreads();
        }
    }
    if (r == 0) {
        float total = 0.f;
        for (uint32_t s = 0; s < nq; ++s) total += loss_s[s];
        a.partial[static_cast<size_t>(member) * a.n_chunks + blockIdx.y] = total;
    }
}

__global__ void k_s2s_finalize(const float* __restrict__ partial, uint32_t P, uint32_t n_chunks, float inv_count,
                               float* __restrict__ fitness)
{
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= P) return;
    float s = 0.f;
    for (uint32_t t = 0; t < n_chunks; ++t) s += partial[static_cast<size_t>(m) * n_chunks + t];
    fitness[m] = -s * inv_count;
}

// ------------------------------------------------------------------------------------------
// tensor-core version (h = 128)
// ------------------------------------------------------------------------------------------
constexpr int kTcH = 128;
constexpr int kTcQ = 128;                                  // queries per block: two halves of 64
constexpr int kTcSub = 1;                                  // warps per TMEM lane quarter and half: each takes 64 / kTcSub queries
constexpr int kTcHalfThreads = 128 * kTcSub;
constexpr int kTcEpiThreads = 2 * kTcHalfThreads;          // half 0's warps first, then half 1's
constexpr int kTcCols = 64 / kTcSub;                       // queries per epilogue thread
constexpr int kTcOutPerThread = kVocab * 64 / kTcHalfThreads;   // read-out: tokens per thread
constexpr int kTcThreads = kTcEpiThreads + 32;             // + the MMA warp
constexpr int kTcKBlocks = 18;                             // K = 128 (h) + 16 (one-hot, 1, padding) in groups of 8
constexpr uint32_t kTcALbo = 64 * 128 + 16;                // 64 row groups of 8 x 16 bytes between K groups, +16 bytes
                                                           // (bank spread of the staging stores)
constexpr uint32_t kTcBLbo = 16 * 128 + 16;                // 16 row groups, +16 bytes so that the 2-byte stores
                                                           // of a warp (4 K groups) fall in distinct banks
constexpr uint32_t kTcABytes = kTcKBlocks * kTcALbo;       // 147,744
constexpr uint32_t kTcBBytes = kTcKBlocks * kTcBLbo;       // 37,152
constexpr uint32_t kTcCellFloats = 4 * kTcH * kVocab + 4 * kTcH * kTcH + 4 * kTcH;   // one LSTM cell

struct __align__(128) S2sSmem {
    unsigned char A[kTcABytes];                            // [Wh | Wx | b | 0] as core matrices
    unsigned char Bop[kTcBBytes];                          // [h; onehot; 1; 0] of the 128 queries
    float oW[16][kVocab][8];                               // read-out weights [K group][token][k], bf16-rounded
    float ob[kVocab];
    float lg[kS2sMaxTd][kTcQ][kVocab];                     // logits of every answer position
    uint8_t enc[kTcQ][kS2sMaxTe + 1], dec[kTcQ][kS2sMaxTd + 1], tgt[kTcQ][kS2sMaxTd + 1];
    float loss_w[kTcThreads / 32];
    uint64_t full[2];                                      // the gates of a half are in TMEM
    uint64_t hready[2];                                    // a half's B operand holds the next step's input
    uint32_t tmem_slot;
    volatile int abort;
};

__device__ __forceinline__ float tanh_sfu(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ bool elect_one()
{
    uint32_t p;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(p));
    return p != 0;
}
// asks the L2 to fetch `bytes` (multiple of 16) starting at a 16-byte aligned address
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(__cvta_generic_to_global(p)), "r"(bytes) : "memory");
}

// One cell's weights -> A operand (all threads of the block).  The rows of the input, forget and
// output gates are halved (exact in bf16) so that their sigma(x) = 0.5 tanh(x / 2) + 0.5 needs no
// scaling of the accumulator.
__device__ __forceinline__ void s2s_stage_weights(S2sSmem& S, const float* __restrict__ cellp, uint32_t tid)
{
    const float* Wx = cellp;
    const float* Wh = Wx + 4 * kTcH * kVocab;
    const float* bb = Wh + 4 * kTcH * kTcH;
    // Wh: 64 groups of 8 rows x 128 k.  A warp reads a whole row with one fully coalesced 128-bit
    // load per lane (lane l gets k = 4l .. 4l+3), 8 rows per group, two groups at a time.  A
    // 16-byte row of a core matrix (8 k) is the data of an even/odd lane pair, so the pair swaps
    // halves: the even lane ends with rows 0-3 of its K group, the odd lane with rows 4-7, and each
    // stores them as 128-bit words (the K-group pitch is padded by 16 bytes so that the four K
    // groups of a quarter-warp fall in distinct banks).
    const uint32_t warp = tid >> 5, lane = tid & 31u;
    const bool odd = lane & 1u;
    constexpr uint32_t kWarps = kTcThreads / 32, G = 2;
#pragma unroll 1
    for (uint32_t mg0 = warp * G; mg0 < 64u; mg0 += kWarps * G) {
        float4 v[G][8];
#pragma unroll
        for (uint32_t g = 0; g < G; ++g)
#pragma unroll
            for (uint32_t r = 0; r < 8u; ++r) {
                const uint32_t mg = min(mg0 + g, 63u);
                v[g][r] = __ldg(reinterpret_cast<const float4*>(Wh + (mg * 8u + r) * kTcH) + lane);
            }
#pragma unroll
        for (uint32_t g = 0; g < G; ++g) {
            const uint32_t mg = mg0 + g;
            if (mg < 64u) {
                const float sc = ((mg >> 4) == 2u) ? 1.0f : 0.5f;       // 16 row groups per gate
                uint32_t w0[8], w1[8];
#pragma unroll
                for (uint32_t r = 0; r < 8u; ++r) {
                    w0[r] = pack_bf16(sc * v[g][r].x, sc * v[g][r].y);
                    w1[r] = pack_bf16(sc * v[g][r].z, sc * v[g][r].w);
                }
                unsigned char* dst = S.A + (lane >> 1) * kTcALbo + mg * 128u + (odd ? 64u : 0u);
#pragma unroll
                for (uint32_t i = 0; i < 4u; ++i) {
                    const uint32_t got0 = __shfl_xor_sync(0xffffffffu, odd ? w0[i] : w0[i + 4], 1);
                    const uint32_t got1 = __shfl_xor_sync(0xffffffffu, odd ? w1[i] : w1[i + 4], 1);
                    const uint32_t keep0 = odd ? w0[i + 4] : w0[i], keep1 = odd ? w1[i + 4] : w1[i];
                    // the even lane's words are k 0-3 of the K group, the odd lane's k 4-7
                    *reinterpret_cast<uint4*>(dst + i * 16u) =
                        odd ? make_uint4(got0, got1, keep0, keep1) : make_uint4(keep0, keep1, got0, got1);
                }
            }
        }
    }
    // K groups 16, 17: Wx[m][0..7] | Wx[m][8..11], b[m], 0, 0, 0
    for (uint32_t m = tid; m < 512u; m += kTcThreads) {
        const float4* wx = reinterpret_cast<const float4*>(Wx + m * kVocab);        // 48-byte rows
        const float4 w0 = __ldg(wx), w1 = __ldg(wx + 1), w2 = __ldg(wx + 2);
        const float sc = ((m >> 7) == 2u) ? 1.0f : 0.5f;
        const float bias = sc * __ldg(bb + m);
        *reinterpret_cast<uint4*>(S.A + 16u * kTcALbo + (m >> 3) * 128u + (m & 7u) * 16u) =
            make_uint4(pack_bf16(sc * w0.x, sc * w0.y), pack_bf16(sc * w0.z, sc * w0.w),
                       pack_bf16(sc * w1.x, sc * w1.y), pack_bf16(sc * w1.z, sc * w1.w));
        *reinterpret_cast<uint4*>(S.A + 17u * kTcALbo + (m >> 3) * 128u + (m & 7u) * 16u) =
            make_uint4(pack_bf16(sc * w2.x, sc * w2.y), pack_bf16(sc * w2.z, sc * w2.w), pack_bf16(bias, 0.f), 0u);
    }
}

// one-hot (+ constant 1) rows of query n for the coming step
__device__ __forceinline__ void s2s_write_onehot(S2sSmem& S, uint32_t n, uint32_t tok)
{
    uint32_t w[8];
    const uint32_t one = (tok & 1u) ? 0x3F800000u : 0x00003F80u;  // bf16 1.0 in the upper / lower half
#pragma unroll
    for (uint32_t i = 0; i < 8u; ++i) w[i] = (i == (tok >> 1)) ? one : 0u;
    w[6] |= 0x00003F80u;                                          // k = 12: the constant input of the bias
    *reinterpret_cast<uint4*>(S.Bop + 16u * kTcBLbo + n * 16u) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(S.Bop + 17u * kTcBLbo + n * 16u) = make_uint4(w[4], w[5], w[6], w[7]);
}

// barrier over the four epilogue warps of one half
__device__ __forceinline__ void half_barrier(uint32_t half)
{
    if (half) asm volatile("bar.sync 2, %0;" :: "n"(kTcHalfThreads) : "memory");
    else      asm volatile("bar.sync 1, %0;" :: "n"(kTcHalfThreads) : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
k_s2s_tc(const S2sArgs a, DeviceStatus* status)
{
    extern __shared__ __align__(128) unsigned char s2s_smem_raw[];
    S2sSmem& S = *reinterpret_cast<S2sSmem*>(s2s_smem_raw);
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31u;
    const uint32_t Te = 2 * a.nd + 1, Td = a.nd + 1, T = Te + Td;
    const uint32_t n_items = a.P * a.n_chunks;
    const PhiloxKey key = philox_key(a.k0, a.k1);

    if (tid == 0) {
        mbar_init(smem_u32(&S.full[0]), 1); mbar_init(smem_u32(&S.full[1]), 1);
        mbar_init(smem_u32(&S.hready[0]), kTcHalfThreads / 32); mbar_init(smem_u32(&S.hready[1]), kTcHalfThreads / 32);
        S.abort = 0;
        mbar_init_fence();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(&S.tmem_slot), 512);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S.tmem_slot;

    uint32_t n_wait = 0u, n_wait1 = 0u;        // completed waits: full[half] (epilogue) / hready[0], hready[1] (MMA warp)
    const bool is_mma = warp >= kTcEpiThreads / 32;
    const uint32_t half = (tid / kTcHalfThreads) & 1u;          // epilogue warps: which 64 queries
    const uint32_t sub = (tid % kTcHalfThreads) >> 7;           // ... and which kTcCols of them
    const uint32_t r = tid & 127u;             // epilogue thread: hidden unit = TMEM lane
    uint32_t staged_chunk = 0xFFFFFFFFu;

    for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const uint32_t member = item / a.n_chunks, chunk = item % a.n_chunks;
        const uint32_t q0 = chunk * kTcQ;
        const uint32_t nq = min(static_cast<uint32_t>(kTcQ), a.B - q0);
        const float* p = a.theta + static_cast<size_t>(member) * a.ldD;

        // ---- per-item setup: queries, zero state, read-out weights, encoder weights ------------
        if (chunk != staged_chunk) {
            if (tid < kTcQ) s2s_query(key, a.status->generation, q0 + min(tid, nq - 1u), a.nd, S.enc[tid], S.dec[tid], S.tgt[tid]);
            staged_chunk = chunk;
        }
        if (is_mma) {                                            // the decoder's weights will be wanted next
            const char* next = reinterpret_cast<const char*>(p + kTcCellFloats);
            constexpr uint32_t piece = kTcCellFloats * 4u / 32u;       // 9,024 bytes per lane
            prefetch_l2(next + lane * piece, piece);
        }
        for (uint32_t i = tid; i < 16u * kTcBLbo / 16u; i += kTcThreads)
            reinterpret_cast<uint4*>(S.Bop)[i] = make_uint4(0u, 0u, 0u, 0u);
        for (uint32_t i = tid; i < kVocab * 16u; i += kTcThreads) {       // (token, K group) -> 8 weights
            const uint32_t o = i >> 4, kb = i & 15u;
            const float4* src = reinterpret_cast<const float4*>(p + 2u * kTcCellFloats + o * kTcH + kb * 8u);
            const float4 w0 = __ldg(src), w1 = __ldg(src + 1);
            float* dst = S.oW[kb][o];
            dst[0] = bf16_round(w0.x); dst[1] = bf16_round(w0.y); dst[2] = bf16_round(w0.z); dst[3] = bf16_round(w0.w);
            dst[4] = bf16_round(w1.x); dst[5] = bf16_round(w1.y); dst[6] = bf16_round(w1.z); dst[7] = bf16_round(w1.w);
        }
        if (tid < kVocab) S.ob[tid] = p[2u * kTcCellFloats + kVocab * kTcH + tid];
        s2s_stage_weights(S, p, tid);
        __syncthreads();                                        // tokens are there
        if (tid < kTcQ) s2s_write_onehot(S, tid, S.enc[tid][0]);
        fence_async_smem();
        __syncthreads();

        float c[kTcCols];
#pragma unroll
        for (int i = 0; i < kTcCols; ++i) c[i] = 0.f;
        float loss = 0.f;

        for (uint32_t phase = 0; phase < 2u; ++phase) {
            const uint32_t t0 = phase ? Te : 0u, t1 = phase ? T : Te;
            if (phase) {
                // every MMA of the encoder has been waited for by an epilogue warp: A may be replaced
                __syncthreads();
                s2s_stage_weights(S, p + kTcCellFloats, tid);
                fence_async_smem();
                __syncthreads();
                if (is_mma && item + gridDim.x < n_items) {     // the next item's encoder cell
                    const uint32_t nm = (item + gridDim.x) / a.n_chunks;
                    const char* next = reinterpret_cast<const char*>(a.theta + static_cast<size_t>(nm) * a.ldD);
                    constexpr uint32_t piece = kTcCellFloats * 4u / 32u;
                    prefetch_l2(next + lane * piece, piece);
                }
            }
            if (is_mma) {
                // ================= MMA warp (the whole warp walks the loop, one lane issues) ===========
                // The halves alternate, so that one half's MMAs run while the other half's gates are
                // being applied.
                constexpr uint32_t idesc = umma_idesc_bf16(128, 64);
                const uint32_t a_base = smem_u32(S.A), b_base = smem_u32(S.Bop);
                for (uint32_t t = t0; t < t1; ++t) {
#pragma unroll
                    for (uint32_t x = 0; x < 2u; ++x) {
                        if (t > 0) {                             // step 0 reads the state the setup wrote
                            uint32_t& n = x ? n_wait1 : n_wait;
                            wait_or_abort(&S.abort, &S.hready[x], n & 1u, status);
                            ++n;
                        }
                        tc_fence_after();
                        if (elect_one()) {
#pragma unroll
                            for (uint32_t g = 0; g < 4u; ++g)
#pragma unroll
                                for (uint32_t kk = 0; kk < kTcKBlocks / 2; ++kk) {
                                    const uint64_t ad = umma_smem_desc(a_base + 2u * kk * kTcALbo + g * 16u * 128u, kTcALbo, 128u);
                                    const uint64_t bd = umma_smem_desc(b_base + 2u * kk * kTcBLbo + x * 8u * 128u, kTcBLbo, 128u);
                                    umma_bf16(tmem + x * 256u + g * 64u, ad, bd, idesc, kk);
                                }
                            umma_commit(smem_u32(&S.full[x]));
                        }
                        __syncwarp();
                    }
                }
            } else {
                // ================= epilogue warps ======================================================
                const uint32_t tq = tmem + (static_cast<uint32_t>((warp & 3u) * 32u) << 16) + half * 256u + sub * kTcCols;
                for (uint32_t t = t0; t < t1; ++t) {
                    wait_or_abort(&S.abort, &S.full[half], n_wait & 1u, status);
                    ++n_wait;
                    tc_fence_after();
                    // chunks of 8 queries; the loads of the next chunk are in flight while this one
                    // is worked on (two register sets)
                    uint32_t g0[2][8], g1[2][8], g2[2][8], g3[2][8];
                    tmem_ld8_issue(tq + 0u * 64u, g0[0]); tmem_ld8_issue(tq + 1u * 64u, g1[0]);
                    tmem_ld8_issue(tq + 2u * 64u, g2[0]); tmem_ld8_issue(tq + 3u * 64u, g3[0]);
                    tmem_ld8x4_fence(g0[0], g1[0], g2[0], g3[0]);
#pragma unroll
                    for (uint32_t ch = 0; ch < kTcCols / 8u; ++ch) {
                        const uint32_t cur = ch & 1u, nxt = cur ^ 1u;
                        if (ch + 1u < kTcCols / 8u) {
                            tmem_ld8_issue(tq + 0u * 64u + (ch + 1u) * 8u, g0[nxt]);
                            tmem_ld8_issue(tq + 1u * 64u + (ch + 1u) * 8u, g1[nxt]);
                            tmem_ld8_issue(tq + 2u * 64u + (ch + 1u) * 8u, g2[nxt]);
                            tmem_ld8_issue(tq + 3u * 64u + (ch + 1u) * 8u, g3[nxt]);
                        }
                        // hidden unit r of query n sits at K group r/8, row n, element r%8
                        unsigned char* dst = S.Bop + (r >> 3) * kTcBLbo + (half * 64u + sub * kTcCols + ch * 8u) * 16u + (r & 7u) * 2u;
#pragma unroll
                        for (int j = 0; j < 8; j += 2) {
                            // the accumulators of the i, f, o gates already hold x / 2
                            float2 hv;
                            {
                                const float ig = fmaf(0.5f, tanh_sfu(__uint_as_float(g0[cur][j])), 0.5f);
                                const float fg = fmaf(0.5f, tanh_sfu(__uint_as_float(g1[cur][j])), 0.5f);
                                const float cg = tanh_sfu(__uint_as_float(g2[cur][j]));
                                const float og = fmaf(0.5f, tanh_sfu(__uint_as_float(g3[cur][j])), 0.5f);
                                float& c0 = c[ch * 8 + j];
                                c0 = fmaf(fg, c0, ig * cg);
                                hv.x = og * tanh_sfu(c0);
                            }
                            {
                                const float ig = fmaf(0.5f, tanh_sfu(__uint_as_float(g0[cur][j + 1])), 0.5f);
                                const float fg = fmaf(0.5f, tanh_sfu(__uint_as_float(g1[cur][j + 1])), 0.5f);
                                const float cg = tanh_sfu(__uint_as_float(g2[cur][j + 1]));
                                const float og = fmaf(0.5f, tanh_sfu(__uint_as_float(g3[cur][j + 1])), 0.5f);
                                float& c1 = c[ch * 8 + j + 1];
                                c1 = fmaf(fg, c1, ig * cg);
                                hv.y = og * tanh_sfu(c1);
                            }
                            const uint32_t hb = pack_bf16(hv.x, hv.y);
                            *reinterpret_cast<uint16_t*>(dst + j * 16) = static_cast<uint16_t>(hb & 0xFFFFu);
                            *reinterpret_cast<uint16_t*>(dst + j * 16 + 16) = static_cast<uint16_t>(hb >> 16);
                        }
                        if (ch + 1u < kTcCols / 8u) tmem_ld8x4_fence(g0[nxt], g1[nxt], g2[nxt], g3[nxt]);
                    }
                    // the coming step's token (none after the last step)
                    if (t + 1u < T && sub == 0u && r < 64u) {
                        const uint32_t n = half * 64u + r;
                        s2s_write_onehot(S, n, (t + 1u < Te) ? S.enc[n][t + 1u] : S.dec[n][t + 1u - Te]);
                    }
                    fence_async_smem();
                    tc_fence_before();
                    if (t >= Te) {
                        // read-out on the CUDA cores from the state just written (all warps of the
                        // half must have written it), while the tensor cores work on the next step
                        half_barrier(half);
                        if (t + 1u < T && lane == 0) mbar_arrive(smem_u32(&S.hready[half]));
                        const uint32_t s = tid & 63u, o0 = ((tid % kTcHalfThreads) >> 6) * kTcOutPerThread;
                        float2 acc[kTcOutPerThread];
#pragma unroll
                        for (int o = 0; o < kTcOutPerThread; ++o) acc[o] = make_float2(0.f, 0.f);
                        const unsigned char* hrow = S.Bop + (half * 64u + s) * 16u;
#pragma unroll 4
                        for (uint32_t kb = 0; kb < 16u; ++kb) {
                            const uint4 hv = *reinterpret_cast<const uint4*>(hrow + kb * kTcBLbo);
                            const uint32_t hw[4] = { hv.x, hv.y, hv.z, hv.w };
                            float2 x[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                x[i] = make_float2(__uint_as_float(hw[i] << 16), __uint_as_float(hw[i] & 0xFFFF0000u));
#pragma unroll
                            for (int o = 0; o < kTcOutPerThread; ++o) {
                                const float4 w0 = *reinterpret_cast<const float4*>(&S.oW[kb][o0 + o][0]);
                                const float4 w1 = *reinterpret_cast<const float4*>(&S.oW[kb][o0 + o][4]);
                                ffma2(acc[o], make_float2(w0.x, w0.y), x[0]);
                                ffma2(acc[o], make_float2(w0.z, w0.w), x[1]);
                                ffma2(acc[o], make_float2(w1.x, w1.y), x[2]);
                                ffma2(acc[o], make_float2(w1.z, w1.w), x[3]);
                            }
                        }
#pragma unroll
                        for (int o = 0; o < kTcOutPerThread; ++o) S.lg[t - Te][half * 64u + s][o0 + o] = (acc[o].x + acc[o].y) + S.ob[o0 + o];
                        // the next epilogue overwrites the state: everyone must be done reading it
                        half_barrier(half);
                    } else {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&S.hready[half]));
                    }
                }
            }
        }
        // ---- the item's loss: cross-entropy of every (position, query), summed in a fixed order ----
        __syncthreads();
        for (uint32_t idx = tid; idx < Td * kTcQ; idx += kTcThreads) {
            const uint32_t pos = idx / kTcQ, q = idx % kTcQ;
            if (q < nq) loss += token_loss(S.lg[pos][q], S.tgt[q][pos]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, off);
        if (lane == 0) S.loss_w[warp] = loss;
        __syncthreads();
        if (tid == 0) {
            float total = 0.f;
            for (int w = 0; w < kTcThreads / 32; ++w) total += S.loss_w[w];
            a.partial[static_cast<size_t>(member) * a.n_chunks + chunk] = total;
        }
        __syncthreads();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
uint32_t s2s_param_count(uint32_t h)
{
    return 2u * (4u * h * kVocab + 4u * h * h + 4u * h) + kVocab * h + kVocab;
}

bool s2s_supported(uint32_t h, uint32_t nd, uint32_t B)
{
    return h >= 32 && h <= 128 && h % 32 == 0 && nd >= 1 && nd <= kS2sMaxDigits && B >= 1;
}

static uint32_t s2s_chunks(uint32_t B, bool tc) { return tc ? (B + kTcQ - 1) / kTcQ : (B + kSimpleQ - 1) / kSimpleQ; }

size_t s2s_scratch_bytes(uint32_t P, uint32_t B)
{
    return static_cast<size_t>(P) * s2s_chunks(B, false) * sizeof(float);     // the finer split bounds both
}

int launch_rollout_s2s(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, uint32_t h, uint32_t nd,
                       uint32_t B, uint32_t k0, uint32_t k1, uint32_t kernel_choice,
                       void* scratch, float* fitness, float* logits, DeviceStatus* status)
{
    const bool want_tc = kernel_choice != EVO_ROLLOUT_GENERIC;
    if (want_tc && (h != kTcH || logits)) {
        if (kernel_choice == EVO_ROLLOUT_TILED) return -2;       // asked for explicitly, not available
    }
    const bool tc = want_tc && h == kTcH && !logits;
    S2sArgs a;
    a.theta = theta; a.ldD = ldD; a.P = P; a.h = h; a.nd = nd; a.B = B;
    a.k0 = k0; a.k1 = k1; a.status = status;
    a.partial = static_cast<float*>(scratch);
    a.n_chunks = s2s_chunks(B, tc);
    a.logits = logits;
    if (tc) {
        static int sm_count = 0;
        if (sm_count == 0) {
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess) return -1;
            if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        }
        if (cudaFuncSetAttribute(k_s2s_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(sizeof(S2sSmem))) != cudaSuccess) return -1;
        const uint32_t items = P * a.n_chunks;
        const uint32_t grid = items < static_cast<uint32_t>(sm_count) ? items : static_cast<uint32_t>(sm_count);
        k_s2s_tc<<<grid, kTcThreads, sizeof(S2sSmem), st>>>(a, status);
    } else {
        dim3 grid(P, a.n_chunks);
        k_s2s_simple<<<grid, 128, 0, st>>>(a);
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    const float inv = 1.0f / (static_cast<float>(B) * static_cast<float>(nd + 1));
    k_s2s_finalize<<<(P + 255u) / 256u, 256, 0, st>>>(a.partial, P, a.n_chunks, inv, fitness);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 2;
}

}  // namespace evo
