// Supervised rollout on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
// The convolutional policy (conv 1->8 5x5, ReLU, pool; conv 8->16 5x5, ReLU, pool; linear
// 256->10) evaluated for every member on the same batch is two dense contractions:
//
//   k_cnn_conv1_tc   conv1 for ALL members at once.  The batch is shared, so the im2col rows
//                    (K = 25 taps padded to 32) are the A operand for every member and the 8P
//                    filters of the population sit side by side on N.  GEMM rows are pooled
//                    pixels; the four conv outputs under a pooling window are four A operands
//                    accumulated into four TMEM column blocks, so the 2x2 max-pool is a max over
//                    registers.  The epilogue adds bias, applies ReLU and writes the pooled
//                    activation as bf16, 8 channels = 16 bytes per pixel.
//   k_cnn_conv2_tc   per member: conv2 as an implicit GEMM with NO im2col copy.  With channels
//                    innermost, the 8 channels of a pixel are one 16-byte row of a UMMA core
//                    matrix, 8 consecutive output columns are 8 consecutive pixels = one 128-byte
//                    core matrix, and the (kh,kw) tap is just an address offset, so the shared
//                    memory descriptors of the A operand point straight into the pooled image
//                    pair that a single bulk copy brought in.  D[128 = 2 images x 8x8][16 filters]
//                    in TMEM; pool, linear layer and cross-entropy on CUDA cores.
//
// Operands are bf16 (round to nearest even), accumulation fp32 in TMEM.  Every wait is bounded:
// on expiry the block records EVO_ERR_TIMEOUT, frees its TMEM and leaves.
// Paper: Section 3 (supervised tasks are single-step tasks; ConvNet on 28x28 images).
#include "internal.h"
#include "async.cuh"
#include "umma.cuh"

namespace evo {

// ------------------------------------------------------------------------------------------
// conv1 for a group of up to 64 members.
//
// GEMM rows are POOLED pixels (128 per tile); the four conv outputs of a 2x2 pooling window are
// four separate A operands (the same 6x6 image patch shifted by (dy,dx)) accumulated into four
// TMEM column blocks, so the max-pool is a max over four registers of one thread, with no
// shuffles.  Unit of work = (tile, 8 members = 64 filters): 8 MMAs (4 windows x K = 2 x 16)
// into one of two 256-column accumulators.  Warp 8 issues the MMAs and runs ahead; warps 0-7 read
// the accumulators (pool, ReLU, bf16; the bias rides in the contraction) and store 16 bytes per
// (member, pixel); warps 9-12 build the next tile's A operands while the epilogues run.
// ------------------------------------------------------------------------------------------
constexpr int kC1EpiThreads = 256;                     // two warps per TMEM lane quarter
constexpr int kC1StageThreads = 128;                   // one thread per pooled pixel of a tile: builds the A operands
constexpr int kC1Threads = kC1EpiThreads + 32 + kC1StageThreads;
constexpr int kC1SmemB = 512 * 32 * 2;                  // all filters of the group, bf16, K = 32
constexpr int kC1SmemAWin = 128 * 32 * 2;               // one window's im2col tile
constexpr int kC1SmemA = 4 * kC1SmemAWin;               // four windows
// the block owns all 512 TMEM columns, so it must be alone on its SM: ask for more than half
// of the SM's shared memory (it uses ~100 KB of it)
constexpr int kC1DynRequest = 120 * 1024;

struct C1Ctl {
    uint64_t a_full[2];          // the A operands of a tile are staged
    uint64_t a_free[2];          // every MMA that read an A buffer has completed
    uint64_t mma_done[2];        // an accumulator is complete
    uint64_t acc_free[2];        // an accumulator has been read out
    uint32_t tmem_slot;
    volatile int abort;
};

// pooled-1 layout: [member][image pair][y 12][image in pair 2][x 12][channel 8] bf16
__device__ __forceinline__ size_t pooled1_offset(uint32_t member, uint32_t n_pairs, uint32_t image,
                                                 uint32_t py, uint32_t px)
{
    return (((static_cast<size_t>(member) * n_pairs + (image >> 1)) * 12 + py) * 2 + (image & 1u)) * 12 + px;
}

// max of three values in one instruction (the 3-input form of max.f32)
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// 6x6 image patch under one pooled pixel (zero for rows past the batch)
__device__ __forceinline__ void c1_load_patch(const float* __restrict__ images, uint32_t gp, uint32_t n_pooled,
                                              float (&patch)[36])
{
    if (gp < n_pooled) {
        const uint32_t img = gp / 144u, rem = gp % 144u, py = rem / 12u, px = rem % 12u;
        const float* src = images + static_cast<size_t>(img) * 784u + (2u * py) * 28u + 2u * px;
#pragma unroll
        for (int r = 0; r < 6; ++r) {
            const float2* row = reinterpret_cast<const float2*>(src + r * 28);     // 2*px is even: 8-byte aligned
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                const float2 v = __ldg(row + c);
                patch[r * 6 + 2 * c] = v.x; patch[r * 6 + 2 * c + 1] = v.y;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 36; ++i) patch[i] = 0.f;
    }
}

// im2col rows of the four windows of pooled pixel `row` into the A buffers (core matrices: 8 rows
// x 16 bytes, k-group kg at +kg*2048, row group at +128)
__device__ __forceinline__ void c1_stage_rows(unsigned char* Abuf, int row, int dy, const float (&patch)[36])
{
#pragma unroll
    for (int dx = 0; dx < 2; ++dx) {                     // the two windows of conv row parity dy
        const int w = 2 * dy + dx;
        uint32_t packed[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int k0 = 2 * k, k1 = 2 * k + 1;
            // taps 25..27 of the padded K = 32 are the constant 1: their weights carry the bias (below)
            const float v0 = (k0 < 25) ? patch[(dy + k0 / 5) * 6 + dx + k0 % 5] : (k0 < 28 ? 1.f : 0.f);
            const float v1 = (k1 < 25) ? patch[(dy + k1 / 5) * 6 + dx + k1 % 5] : (k1 < 28 ? 1.f : 0.f);
            packed[k] = pack_bf16(v0, v1);
        }
#pragma unroll
        for (int kg = 0; kg < 4; ++kg)
            *reinterpret_cast<uint4*>(Abuf + w * kC1SmemAWin + (kg * 16 + (row >> 3)) * 128 + (row & 7) * 16) =
                make_uint4(packed[4 * kg], packed[4 * kg + 1], packed[4 * kg + 2], packed[4 * kg + 3]);
    }
}

__global__ void __launch_bounds__(kC1Threads, 1)
k_cnn_conv1_tc(const float* __restrict__ theta, uint32_t ldD, uint32_t P, const float* __restrict__ images,
               uint32_t batch, uint4* __restrict__ pooled1, uint32_t* work_counter, DeviceStatus* status)
{
    extern __shared__ __align__(1024) unsigned char dyn[];
    __shared__ __align__(8) C1Ctl ctl;

    unsigned char* Bsm = dyn;                                           // 32 KB
    unsigned char* Asm = dyn + kC1SmemB;                                // 2 x 32 KB

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t group0 = blockIdx.y * 64u;                           // first member of this block's group
    const uint32_t n_members = min(64u, P - group0);
    const uint32_t n_gm = (n_members + 7u) / 8u;                        // units per tile
    const uint32_t n_pairs = (batch + 1u) / 2u;
    const uint32_t n_pooled = batch * 144u;
    const uint32_t n_tiles = (n_pooled + 127u) / 128u;

    if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) *work_counter = 0;   // for the conv2 kernel

    // ---- B operand: W1 of every member of the group, [filter][k] -> core matrices (k-group, member)
    for (uint32_t idx = tid; idx < 512u * 4u; idx += kC1Threads) {
        const uint32_t f = idx >> 2, kg = idx & 3u;                     // filter, 8-tap group
        const uint32_t m = f >> 3, ch = f & 7u;
        uint32_t w[4] = { 0, 0, 0, 0 };
        if (m < n_members) {
            const float* src = theta + static_cast<size_t>(group0 + m) * ldD + ch * 25u + kg * 8u;
            // The bias rides in the contraction: against the three constant-1 taps stand three bf16 pieces of
            // it, b = b0 + b1 + b2 to 24 bits, so the fp32 accumulator starts from the unrounded bias and
            // the epilogue has nothing to add.
            const float b = theta[static_cast<size_t>(group0 + m) * ldD + 200u + ch];
            const float b0 = __bfloat162float(__float2bfloat16_rn(b));
            const float b1 = __bfloat162float(__float2bfloat16_rn(b - b0));
            const float b2 = (b - b0) - b1;
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t kk = kg * 8u + k;
                v[k] = kk < 25u ? src[k] : (kk == 25u ? b0 : (kk == 26u ? b1 : (kk == 27u ? b2 : 0.f)));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) w[k] = pack_bf16(v[2 * k], v[2 * k + 1]);
        }
        *reinterpret_cast<uint4*>(Bsm + (kg * 64u + (f >> 3)) * 128u + (f & 7u) * 16u) = make_uint4(w[0], w[1], w[2], w[3]);
    }

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&ctl.a_full[i]), 1);
            mbar_init(smem_u32(&ctl.a_free[i]), 1);
            mbar_init(smem_u32(&ctl.mma_done[i]), 1);
            mbar_init(smem_u32(&ctl.acc_free[i]), kC1EpiThreads / 32);
        }
        ctl.abort = 0;
        mbar_init_fence();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(&ctl.tmem_slot), 512);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl.tmem_slot;

    if (warp == kC1EpiThreads / 32) {
        // ================= MMA issuer =============================================================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, 64);
            const uint32_t a_base = smem_u32(Asm), b_base = smem_u32(Bsm);
            uint32_t u = 0, ti = 0;
            for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++ti) {
                wait_or_abort(&ctl.abort, &ctl.a_full[ti & 1u], (ti >> 1) & 1u, status);
                const uint32_t a0 = a_base + (ti & 1u) * kC1SmemA;
                for (uint32_t gm = 0; gm < n_gm; ++gm, ++u) {
                    const uint32_t buf = u & 1u;
                    wait_or_abort(&ctl.abort, &ctl.acc_free[buf], (u >> 1) & 1u, status);
                    tc_fence_after();
#pragma unroll
                    for (uint32_t w = 0; w < 4u; ++w)
#pragma unroll
                        for (uint32_t ks = 0; ks < 2u; ++ks) {
                            const uint64_t ad = umma_smem_desc(a0 + w * kC1SmemAWin + ks * 2u * 2048u, 2048u, 128u);
                            const uint64_t bd = umma_smem_desc(b_base + ks * 2u * 8192u + gm * 8u * 128u, 8192u, 128u);
                            umma_bf16(tmem + buf * 256u + w * 64u, ad, bd, idesc, ks);
                        }
                    umma_commit(smem_u32(&ctl.mma_done[buf]));
                }
                umma_commit(smem_u32(&ctl.a_free[ti & 1u]));       // arrives once this tile's MMAs are done
            }
        }
    } else if (warp > kC1EpiThreads / 32) {
        // ================= staging warps: im2col rows of the tiles, one tile ahead of the MMAs ============
        // thread = pooled pixel of the tile; the 6x6 image patch under it gives the rows of all four
        // pooling windows.  The buffer of tile ti is free once the MMAs of tile ti - 2 have completed.
        const int row = tid - (kC1EpiThreads + 32);
        float patch[36];
        uint32_t ti = 0;
        for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++ti) {
            c1_load_patch(images, tile * 128u + row, n_pooled, patch);
            if (ti >= 2u) wait_or_abort(&ctl.abort, &ctl.a_free[ti & 1u], ((ti >> 1) - 1u) & 1u, status);
            unsigned char* Abuf = Asm + (ti & 1u) * kC1SmemA;
            c1_stage_rows(Abuf, row, 0, patch);
            c1_stage_rows(Abuf, row, 1, patch);
            fence_async_smem();
            asm volatile("bar.sync 2, %0;" :: "n"(kC1StageThreads) : "memory");
            if (row == 0) mbar_arrive(smem_u32(&ctl.a_full[ti & 1u]));
        }
        // the last arrivals on a_free land in this block's shared memory: see them in before the block ends
        if (row < 2 && ti > static_cast<uint32_t>(row)) {
            const uint32_t n_done = (ti - row + 1u) >> 1;              // completions of buffer `row`
            wait_or_abort(&ctl.abort, &ctl.a_free[row], (n_done - 1u) & 1u, status);
        }
    } else {
        // ================= epilogue warps ==========================================================
        if (lane == 0) { mbar_arrive(smem_u32(&ctl.acc_free[0])); mbar_arrive(smem_u32(&ctl.acc_free[1])); }
        const int row = tid & 127, half = tid >> 7;       // my pooled pixel (= TMEM lane) and my half of the members
        uint32_t u = 0, ti = 0;
        for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++ti) {
            const uint32_t gp = tile * 128u + row;                     // my pooled pixel = my TMEM lane
            const bool pix_ok = gp < n_pooled;
            const uint32_t img = gp / 144u, rem = gp % 144u, py = rem / 12u, px = rem % 12u;
            const size_t pix_off = pooled1_offset(0u, n_pairs, img, py, px);     // + member * member_stride
            const size_t member_stride = static_cast<size_t>(n_pairs) * (12u * 2u * 12u);

            for (uint32_t gm = 0; gm < n_gm; ++gm, ++u) {
                const uint32_t buf = u & 1u;
                wait_or_abort(&ctl.abort, &ctl.mma_done[buf], (u >> 1) & 1u, status);
                tc_fence_after();
                const uint32_t t0 = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16) + buf * 256u + half * 32u;
                // My four members of the unit, one at a time: the 8 filters of a member under the four
                // pooling windows are 4 x 8 columns.  The loads of the next member are in flight while
                // this one is pooled and stored (two register buffers).
                uint32_t ra[4][8], rb[4][8];
#pragma unroll
                for (int w = 0; w < 4; ++w) tmem_ld8_issue(t0 + w * 64u, ra[w]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t (&cur)[4][8] = (j & 1) ? rb : ra;
                    uint32_t (&nxt)[4][8] = (j & 1) ? ra : rb;
                    tmem_ld8x4_fence(cur[0], cur[1], cur[2], cur[3]);
                    if (j < 3) {
#pragma unroll
                        for (int w = 0; w < 4; ++w) tmem_ld8_issue(t0 + w * 64u + (j + 1) * 8u, nxt[w]);
                    } else {                                             // my part of the accumulator is in registers
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctl.acc_free[buf]));
                    }
                    const uint32_t m = gm * 8u + half * 4u + j;
                    // the accumulators already contain the bias: relu(max4) = two 3-input max per value
                    uint32_t o[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float v[2];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int k = 2 * c + h;
                            const float m3 = fmax3(__uint_as_float(cur[0][k]), __uint_as_float(cur[1][k]), __uint_as_float(cur[2][k]));
                            v[h] = fmax3(m3, __uint_as_float(cur[3][k]), 0.f);
                        }
                        o[c] = pack_bf16(v[0], v[1]);
                    }
                    if (pix_ok && m < n_members)
                        pooled1[pix_off + static_cast<size_t>(group0 + m) * member_stride] = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------
// conv2 + pool + linear + cross-entropy, one work item = (member, 16 image pairs).
// Warp-specialised: warp 4 only issues tensor-core work (13 MMAs per image pair, running ahead
// of the epilogue through two 16-column TMEM accumulators); warps 0-3 take the accumulators out
// of TMEM (pool, bias, ReLU), keep the pooled activations of the item's 32 images in shared
// memory and run the linear layer and the cross-entropy once per item.  Pooled image pairs
// arrive through a 4-deep ring of bulk copies.  The roles meet only on mbarriers; every wait is
// bounded, and after a time-out all later waits fall through so that no role is left behind.
// ------------------------------------------------------------------------------------------
constexpr int kC2EpiThreads = 128;
constexpr int kC2Threads = kC2EpiThreads + 32;
constexpr int kPairsPerItem = 16;
constexpr uint32_t kPairBytes = 12 * 2 * 12 * 16;        // 4608
constexpr int kC2Bufs = 4;
constexpr int kP2Stride = 258;                           // bf16 elements; 129 words: image rows fall in distinct banks
constexpr uint32_t kNoItem = 0xFFFFFFFFu;

struct __align__(128) C2Smem {
    unsigned char a[kC2Bufs][kPairBytes];                // pooled image pairs (ring)
    unsigned char b[26 * 2 * 128];                       // W2 as core matrices (tap, filter group)
    float wfT[256 * 12];                                 // linear layer transposed [k][class], bf16-rounded
    __align__(16) __nv_bfloat16 p2[2 * kPairsPerItem][kP2Stride];   // pooled-2 activations of the item's images (they are
                                                         // bf16 operands of the linear layer anyway; half the size lets
                                                         // four blocks share an SM)
    float logit[2 * kPairsPerItem][12];
    float b2[16];
    float bfc[12];
    uint64_t full[kC2Bufs];                              // a ring slot has landed
    uint64_t mma_done[2];                                // an accumulator is complete
    uint64_t acc_free[2];                                // an accumulator has been read out
    uint64_t item_ready;                                 // weights of the next item are staged
    uint32_t tmem_slot;
    volatile int abort;
    volatile uint32_t item;
    volatile int n;
};

__device__ __forceinline__ void c2_wait(C2Smem& S, uint64_t* bar, uint32_t parity, DeviceStatus* status)
{
    wait_or_abort(&S.abort, bar, parity, status);
}

__device__ __forceinline__ void c2_load_pair(C2Smem& S, int buf, const unsigned char* src)
{
    bulk_copy_g2s(smem_u32(S.a[buf]), src, kPairBytes, smem_u32(&S.full[buf]));
}

// 13 MMAs (K = 16 each = two 5x5 taps x 8 channels) of one image pair into one accumulator.
// Tap g = (kh, kw) of the A operand is the pooled pair shifted by kh rows (384 B) and kw pixels
// (16 B); the loop is unrolled so that all offsets are immediates.
__device__ __forceinline__ void c2_issue_mma(uint32_t a0, uint32_t b0, uint32_t d_tmem, uint32_t bar)
{
    constexpr uint32_t idesc = umma_idesc_bf16(128, 16);
#pragma unroll
    for (uint32_t j = 0; j < 13u; ++j) {
        const uint32_t g0 = 2u * j, g1 = 2u * j + 1u;
        const uint32_t off0 = (g0 / 5u) * 384u + (g0 % 5u) * 16u;
        const uint32_t off1 = (g1 < 25u) ? (g1 / 5u) * 384u + (g1 % 5u) * 16u : off0;   // tap 25 = zero weights
        const uint64_t ad = umma_smem_desc(a0 + off0, off1 - off0, 192u);
        const uint64_t bd = umma_smem_desc(b0 + j * 512u, 256u, 128u);
        umma_bf16(d_tmem, ad, bd, idesc, j);
    }
    umma_commit(bar);
}

__global__ void __launch_bounds__(kC2Threads)
k_cnn_conv2_tc(const float* __restrict__ theta, uint32_t ldD, uint32_t P, const unsigned char* __restrict__ pooled1,
               const int32_t* __restrict__ labels, uint32_t batch,
               float* __restrict__ loss, uint32_t* work_counter, DeviceStatus* status)
{
    extern __shared__ __align__(1024) unsigned char dyn[];
    C2Smem& S = *reinterpret_cast<C2Smem*>(dyn);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_pairs = (batch + 1u) / 2u;
    const uint64_t n_units = static_cast<uint64_t>(P) * n_pairs;      // (member, image pair), member-major

    if (tid == 0) {
        for (int i = 0; i < kC2Bufs; ++i) mbar_init(smem_u32(&S.full[i]), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&S.mma_done[i]), 1); mbar_init(smem_u32(&S.acc_free[i]), 4); }
        mbar_init(smem_u32(&S.item_ready), 1);
        S.abort = 0;
        mbar_init_fence();
    }
    for (int k = tid; k < 256; k += kC2Threads) { S.wfT[k * 12 + 10] = 0.f; S.wfT[k * 12 + 11] = 0.f; }
    if (tid < 2) S.bfc[10 + tid] = 0.f;
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(&S.tmem_slot), 32);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = S.tmem_slot;

    if (warp == 4) {
        // ================= MMA issuer: one thread, runs ahead of the epilogue =================
        if (lane == 0) {
            uint32_t gp = 0, item_par = 0, full_par = 0, free_par = 0;
            const uint32_t b0 = smem_u32(S.b);
            for (;;) {
                c2_wait(S, &S.item_ready, item_par, status);
                item_par ^= 1u;
                if (S.item == kNoItem || S.abort) break;
                const int n = S.n;
                for (int i = 0; i < n; ++i, ++gp) {
                    const uint32_t slot = gp % kC2Bufs, acc = gp & 1u;
                    c2_wait(S, &S.full[slot], (full_par >> slot) & 1u, status);
                    full_par ^= (1u << slot);
                    c2_wait(S, &S.acc_free[acc], (free_par >> acc) & 1u, status);
                    free_par ^= (1u << acc);
                    tc_fence_after();
                    c2_issue_mma(smem_u32(S.a[slot]), b0, tmem + 16u * acc, smem_u32(&S.mma_done[acc]));
                }
            }
        }
    } else {
        // ================= epilogue warps ========================================================
        // both accumulators start out free
        if (lane == 0) { mbar_arrive(smem_u32(&S.acc_free[0])); mbar_arrive(smem_u32(&S.acc_free[1])); }
        uint32_t gp = 0, done_par = 0;
        // Image pairs are equal in cost, so every block takes one contiguous range of (member, pair)
        // units, equal to within one pair, and walks it in items of up to 16 pairs of one member:
        // consecutive items belong to the same member almost always, and a member's weights are
        // staged only when the member changes.  The loss is written per image, so the result does
        // not depend on where the ranges are cut.
        const uint32_t unit_end = static_cast<uint32_t>((static_cast<uint64_t>(blockIdx.x) + 1u) * n_units / gridDim.x);
        uint32_t staged_member = 0xFFFFFFFFu;
        uint32_t next = static_cast<uint32_t>(static_cast<uint64_t>(blockIdx.x) * n_units / gridDim.x);
        for (;;) {
            if (tid == 0)                            // one thread decides, so the whole team takes one branch
                S.item = (S.abort || next >= unit_end) ? kNoItem : next;
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
            const uint32_t item = S.item;
            if (item == kNoItem) break;
            const uint32_t member = item / n_pairs;
            const uint32_t pair0 = item % n_pairs;
            const int n = static_cast<int>(min(min(n_pairs - pair0, unit_end - item), static_cast<uint32_t>(kPairsPerItem)));
            next = item + static_cast<uint32_t>(n);
            const int n_img = static_cast<int>(min(batch, 2u * (pair0 + n)) - 2u * pair0);
            const float* prm = theta + static_cast<size_t>(member) * ldD;
            const unsigned char* src = pooled1 + (static_cast<size_t>(member) * n_pairs + pair0) * kPairBytes;

            // every earlier pair has been consumed (its accumulator was waited for), so the ring is free
            if (tid == 0)
                for (int i = 0; i < min(kC2Bufs, n); ++i)
                    c2_load_pair(S, (gp + i) % kC2Bufs, src + static_cast<size_t>(i) * kPairBytes);

            // ---- weights: coalesced reads, then the operand layouts are built from shared memory ----
            float* raw = reinterpret_cast<float*>(&S.p2[0][0]);     // 3,200 floats of scratch
            static_assert(sizeof(S.p2) >= 3200 * sizeof(float), "weight scratch fits in the activation buffer");
            if (member != staged_member) {
            staged_member = member;
            {   // conv2 weights (offset 208) and linear weights (offset 3424) start 16-byte aligned
                const float4* w2v = reinterpret_cast<const float4*>(prm + 208u);
                const float4* wfv = reinterpret_cast<const float4*>(prm + 3424u);
                float4 t2[7], tf[5];
#pragma unroll
                for (int k = 0; k < 7; ++k) t2[k] = (tid + k * kC2EpiThreads < 800) ? __ldg(w2v + tid + k * kC2EpiThreads) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int k = 0; k < 5; ++k) tf[k] = __ldg(wfv + tid + k * kC2EpiThreads);
#pragma unroll
                for (int k = 0; k < 7; ++k)
                    if (tid + k * kC2EpiThreads < 800) reinterpret_cast<float4*>(raw)[tid + k * kC2EpiThreads] = t2[k];
#pragma unroll
                for (int k = 0; k < 5; ++k) {
                    // flat index cls*256 + (c*16 + pos), 4 consecutive pos; stored at row pos*16 + c
                    const uint32_t i = 4u * (tid + k * kC2EpiThreads);
                    const uint32_t cls = i >> 8, c = (i >> 4) & 15u, pos = i & 15u;
                    float* d = S.wfT + (pos * 16u + c) * 12u + cls;
                    d[0 * 192]  = __bfloat162float(__float2bfloat16_rn(tf[k].x));
                    d[1 * 192]  = __bfloat162float(__float2bfloat16_rn(tf[k].y));
                    d[2 * 192]  = __bfloat162float(__float2bfloat16_rn(tf[k].z));
                    d[3 * 192]  = __bfloat162float(__float2bfloat16_rn(tf[k].w));
                }
            }
            if (tid < 16) S.b2[tid] = prm[3408u + tid];
            if (tid < 10) S.bfc[tid] = prm[5984u + tid];
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
            // W2[oc][ic][kh][kw] -> k = (kh*5+kw)*8 + ic: core matrix (tap g, oc/8), row oc%8, 16 bytes = 8 ic
            for (uint32_t idx = tid; idx < 26u * 16u; idx += kC2EpiThreads) {
                const uint32_t g = idx >> 4, oc = idx & 15u;
                uint32_t w[4] = { 0, 0, 0, 0 };
                if (g < 25u) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        w[k] = pack_bf16(raw[(oc * 8u + 2 * k) * 25u + g], raw[(oc * 8u + 2 * k + 1) * 25u + g]);
                }
                *reinterpret_cast<uint4*>(S.b + (g * 2u + (oc >> 3)) * 128u + (oc & 7u) * 16u) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            fence_async_smem();
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
            }
            if (tid == 0) { S.n = n; __threadfence_block(); mbar_arrive(smem_u32(&S.item_ready)); }

            // After the 2x2 max (lanes ^1 = x parity, ^16 = y parity) done as a reduce-scatter, this
            // lane owns channels c0..c0+3 of pooled pixel (image im, row py = warp, column px).
            const int c0 = 8 * (lane & 1) + 4 * ((lane >> 4) & 1);
            const int im = (lane >> 3) & 1, px = (lane & 7) >> 1, py = warp;
            float bias4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) bias4[j] = S.b2[c0 + j];

            for (int i = 0; i < n; ++i, ++gp) {
                const uint32_t slot = gp % kC2Bufs, acc = gp & 1u;
                c2_wait(S, &S.mma_done[acc], (done_par >> acc) & 1u, status);
                done_par ^= (1u << acc);
                tc_fence_after();
                // pair i has been consumed by the tensor core: its ring slot takes pair i + ring depth
                if (tid == 0 && i + kC2Bufs < n) c2_load_pair(S, slot, src + static_cast<size_t>(i + kC2Bufs) * kPairBytes);
                // lane = (y%2, image, x); 2x2 max = lanes ^1 and ^16; + bias, ReLU, bf16
                float r[16];
                tmem_ld16(tmem + (static_cast<uint32_t>(warp * 32) << 16) + 16u * acc, r);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&S.acc_free[acc]));   // values are in registers now
                {
                    const bool up0 = lane & 1, up1 = lane & 16;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float keep = up0 ? r[8 + c] : r[c];
                        const float give = up0 ? r[c] : r[8 + c];
                        r[c] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, give, 1));
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float keep = up1 ? r[4 + c] : r[c];
                        const float give = up1 ? r[c] : r[4 + c];
                        r[c] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, give, 16));
                    }
                    // activation index inside the item: (pixel, channel), channel innermost
                    uint32_t* dst = reinterpret_cast<uint32_t*>(&S.p2[2 * i + im][(py * 4 + px) * 16 + c0]);
                    dst[0] = pack_bf16(fmaxf(r[0] + bias4[0], 0.f), fmaxf(r[1] + bias4[1], 0.f));
                    dst[1] = pack_bf16(fmaxf(r[2] + bias4[2], 0.f), fmaxf(r[3] + bias4[3], 0.f));
                }
            }
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");

            // ---- linear 256 -> 10 for all images of the item: thread = (image, quarter of the inputs);
            //      the partial logits meet in the ring buffers, which are idle now ----
            float* part = reinterpret_cast<float*>(S.a[0]);            // [4][32][12]
            {
                float acc[12];
#pragma unroll
                for (int j = 0; j < 12; ++j) acc[j] = 0.f;
                if (lane < 2 * n) {
                    const uint32_t* x2 = reinterpret_cast<const uint32_t*>(&S.p2[lane][64 * warp]);   // two inputs per word
                    const float* wr = S.wfT + 64 * warp * 12;
#pragma unroll 2
                    for (int k2 = 0; k2 < 32; ++k2) {
                        const uint32_t pair = x2[k2];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const float xv = __uint_as_float(h ? (pair & 0xFFFF0000u) : (pair << 16));
                            const float* wk = wr + (2 * k2 + h) * 12;
                            const float4 w0 = *reinterpret_cast<const float4*>(wk);
                            const float4 w1 = *reinterpret_cast<const float4*>(wk + 4);
                            const float4 w2 = *reinterpret_cast<const float4*>(wk + 8);
                            acc[0] = fmaf(w0.x, xv, acc[0]); acc[1] = fmaf(w0.y, xv, acc[1]);
                            acc[2] = fmaf(w0.z, xv, acc[2]); acc[3] = fmaf(w0.w, xv, acc[3]);
                            acc[4] = fmaf(w1.x, xv, acc[4]); acc[5] = fmaf(w1.y, xv, acc[5]);
                            acc[6] = fmaf(w1.z, xv, acc[6]); acc[7] = fmaf(w1.w, xv, acc[7]);
                            acc[8] = fmaf(w2.x, xv, acc[8]); acc[9] = fmaf(w2.y, xv, acc[9]);
                        }
                    }
                }
                float4* pw = reinterpret_cast<float4*>(part + (warp * 32 + lane) * 12);
                pw[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                pw[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                pw[2] = make_float4(acc[8], acc[9], 0.f, 0.f);
            }
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
            for (int o = tid; o < 32 * 12; o += kC2EpiThreads)          // quarters added in a fixed order
                S.logit[o / 12][o % 12] = ((part[o] + part[384 + o]) + (part[768 + o] + part[1152 + o])) + S.bfc[o % 12];
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
            if (warp == 0) {
                float l = 0.f;
                if (lane < n_img) {
                    const float* lg = S.logit[lane];
                    float mx = lg[0];
#pragma unroll
                    for (int k = 1; k < 10; ++k) mx = fmaxf(mx, lg[k]);
                    float se = 0.f;
#pragma unroll
                    for (int k = 0; k < 10; ++k) se += expf(lg[k] - mx);
                    const int lab = min(max(labels[2u * pair0 + lane], 0), 9);
                    l = (mx + logf(se)) - lg[lab];
                }
                // after a time-out the numbers mean nothing: NaN, which makes tell skip the update
                if (lane < n_img)
                    loss[static_cast<size_t>(member) * batch + 2u * pair0 + lane] = S.abort ? __int_as_float(0x7FC00000) : l;
            }
            fence_async_smem();        // the ring buffers held partial logits; bulk copies write them next
            asm volatile("bar.sync 1, %0;" :: "n"(kC2EpiThreads) : "memory");
        }
        // release the issuer
        if (tid == 0) { S.item = kNoItem; __threadfence_block(); mbar_arrive(smem_u32(&S.item_ready)); }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 32);
}

// fitness[m] = -mean over the batch of the per-image losses: one block per member, fixed order
// (thread t adds images t, t + 256, ...; then a tree over the threads)
__global__ void __launch_bounds__(256)
k_cnn_tc_finalize(const float* __restrict__ loss, uint32_t batch, float* __restrict__ fitness)
{
    __shared__ float red[256];
    const uint32_t m = blockIdx.x;
    float s = 0.f;
    for (uint32_t i = threadIdx.x; i < batch; i += 256u) s += loss[static_cast<size_t>(m) * batch + i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (uint32_t off = 128u; off > 0u; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) fitness[m] = -red[0] / static_cast<float>(batch);
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
size_t cnn_tc_scratch_bytes(uint32_t P, uint32_t batch)
{
    const size_t n_pairs = (batch + 1u) / 2u;
    size_t b = 256;                                                        // work counter
    b += (static_cast<size_t>(P) * batch * sizeof(float) + 255) / 256 * 256;      // per-image losses
    b += static_cast<size_t>(P) * n_pairs * kPairBytes;
    return b;
}

int launch_rollout_cnn_tc(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, const float* images,
                          const int32_t* labels, uint32_t batch, void* scratch, float* fitness,
                          DeviceStatus* status)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return -1;
        if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    }
    unsigned char* base = static_cast<unsigned char*>(scratch);
    uint32_t* counter = reinterpret_cast<uint32_t*>(base);
    float* loss = reinterpret_cast<float*>(base + 256);
    unsigned char* pooled1 = base + 256 + (static_cast<size_t>(P) * batch * sizeof(float) + 255) / 256 * 256;

    if (cudaFuncSetAttribute(k_cnn_conv1_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kC1DynRequest) != cudaSuccess) return -1;
    const uint32_t n_tiles = (batch * 144u + 127u) / 128u;
    dim3 g1(min(static_cast<uint32_t>(sm_count), n_tiles), (P + 63u) / 64u);
    k_cnn_conv1_tc<<<g1, kC1Threads, kC1DynRequest, st>>>(theta, ldD, P, images, batch,
                                                          reinterpret_cast<uint4*>(pooled1), counter, status);
    if (cudaGetLastError() != cudaSuccess) return -1;

    const int c2_bytes = static_cast<int>(sizeof(C2Smem));
    if (cudaFuncSetAttribute(k_cnn_conv2_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, c2_bytes) != cudaSuccess) return -1;
    const uint64_t n_units = static_cast<uint64_t>(P) * ((batch + 1u) / 2u);
    const uint32_t g2 = static_cast<uint32_t>(min(n_units, static_cast<uint64_t>(sm_count) * 4u));   // 4 blocks of ~55 KB per SM
    k_cnn_conv2_tc<<<g2, kC2Threads, c2_bytes, st>>>(theta, ldD, P, pooled1, labels, batch, loss, counter, status);
    if (cudaGetLastError() != cudaSuccess) return -1;
    k_cnn_tc_finalize<<<P, 256, 0, st>>>(loss, batch, fitness);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 3;
}

}  // namespace evo
