// Triangle-painting task (paper Section 3, "Concrete and Abstract Painting"): a member is N
// semi-transparent triangles, fitness = minus the mean squared distance between the painted canvas
// and a target image.  The solver is used on its own here (no policy network): the parameter row IS
// the painting.
//
// Conventions: 10 numbers per triangle (x0 y0 x1 y1 x2 y2 r g b a), each mapped to the unit interval
// by u = clamp(0.5 + 0.5 v, 0, 1); canvas = unit square sampled at pixel centres, starting at a
// grey background; triangles composited in order, C <- C + a (c - C).  Which pixels a triangle
// covers is decided in fp32 with singly rounded operations (explicit *_rn intrinsics: no fused
// contraction), so that the decision is the same on every conforming machine: the pixel centre lies
// in the closed bounding box of the vertices and the three edge values
// e = (bx - ax)(py - ay) - (by - ay)(px - ax) are all >= 0 or all <= 0; a triangle without area
// paints nothing.
//
// k_paint: block = (member, 32 x 16 pixel tile), thread = 4 horizontally adjacent pixels with their
// colours in registers.  The block first turns the member's parameters into triangle records in
// shared memory and drops the triangles whose bounding box misses the tile; the pixel loop then
// walks the surviving records (broadcast shared-memory loads).  Plain fp32 arithmetic.
#include "internal.h"

namespace evo {

constexpr int kPaintThreads = 128;
constexpr int kPaintTileW = 32, kPaintTileH = 16;
constexpr int kPaintMaxTriangles = 512;

struct PaintTri {                 // 16 floats
    float x0, y0, x1, y1, x2, y2;
    float r, g, b, a;
    float xmin, xmax, ymin, ymax;
    float pad0, pad1;
};

__device__ __forceinline__ float paint_unit(float v)
{
    float u = __fmaf_rn(0.5f, v, 0.5f);
    u = (u >= 0.0f) ? u : 0.0f;               // NaN -> 0
    return fminf(u, 1.0f);
}

__device__ __forceinline__ float paint_edge(float ax, float ay, float bx, float by, float px, float py)
{
    const float dx = __fsub_rn(bx, ax), dy = __fsub_rn(by, ay);
    const float qx = __fsub_rn(px, ax), qy = __fsub_rn(py, ay);
    return __fsub_rn(__fmul_rn(dx, qy), __fmul_rn(dy, qx));
}

struct PaintArgs {
    const float* theta; uint32_t ldD, P;
    uint32_t n_tri, W, H;
    float background;
    const float* target;          // [H][W][3]
    float* partial;               // [P][tiles] sums of squared differences
    float* canvas;                // nullable: [P][H][W][3]
    uint32_t tiles_x, tiles_y;
};

__global__ void __launch_bounds__(kPaintThreads)
k_paint(const PaintArgs a)
{
    // sized by the launch: n_tri records, then n_tri indices of the triangles that touch the tile, in order
    extern __shared__ __align__(16) unsigned char paint_smem[];
    PaintTri* tri = reinterpret_cast<PaintTri*>(paint_smem);
    uint16_t* keep = reinterpret_cast<uint16_t*>(paint_smem + sizeof(PaintTri) * a.n_tri);
    __shared__ uint32_t n_keep;
    __shared__ uint32_t warp_count[kPaintThreads / 32];
    __shared__ float warp_sum[kPaintThreads / 32];

    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t member = blockIdx.x, tile = blockIdx.y;
    const uint32_t tx = tile % a.tiles_x, ty = tile / a.tiles_x;
    const float inv_w = __fdiv_rn(1.0f, static_cast<float>(a.W)), inv_h = __fdiv_rn(1.0f, static_cast<float>(a.H));
    const uint32_t i0 = tx * kPaintTileW, j0 = ty * kPaintTileH;
    const uint32_t i1 = min(i0 + kPaintTileW, a.W) - 1u, j1 = min(j0 + kPaintTileH, a.H) - 1u;
    // pixel centres covered by the tile
    const float tile_x0 = __fmul_rn(__fadd_rn(static_cast<float>(i0), 0.5f), inv_w);
    const float tile_x1 = __fmul_rn(__fadd_rn(static_cast<float>(i1), 0.5f), inv_w);
    const float tile_y0 = __fmul_rn(__fadd_rn(static_cast<float>(j0), 0.5f), inv_h);
    const float tile_y1 = __fmul_rn(__fadd_rn(static_cast<float>(j1), 0.5f), inv_h);
    const float* p = a.theta + static_cast<size_t>(member) * a.ldD;

    // ---- triangle records; ordered list of those that can touch the tile ----------------------
    if (tid == 0) n_keep = 0u;
    __syncthreads();
    for (uint32_t base = 0; base < a.n_tri; base += kPaintThreads) {
        const uint32_t k = base + tid;
        bool touches = false;
        if (k < a.n_tri) {
            const float2* src = reinterpret_cast<const float2*>(p + k * 10u);     // 40-byte records
            const float2 v0 = __ldg(src), v1 = __ldg(src + 1), v2 = __ldg(src + 2), v3 = __ldg(src + 3), v4 = __ldg(src + 4);
            PaintTri t;
            t.x0 = paint_unit(v0.x); t.y0 = paint_unit(v0.y);
            t.x1 = paint_unit(v1.x); t.y1 = paint_unit(v1.y);
            t.x2 = paint_unit(v2.x); t.y2 = paint_unit(v2.y);
            t.r = paint_unit(v3.x); t.g = paint_unit(v3.y); t.b = paint_unit(v4.x); t.a = paint_unit(v4.y);
            t.xmin = fminf(t.x0, fminf(t.x1, t.x2)); t.xmax = fmaxf(t.x0, fmaxf(t.x1, t.x2));
            t.ymin = fminf(t.y0, fminf(t.y1, t.y2)); t.ymax = fmaxf(t.y0, fmaxf(t.y1, t.y2));
            t.pad0 = 0.f; t.pad1 = 0.f;
            tri[k] = t;
            const bool has_area = paint_edge(t.x0, t.y0, t.x1, t.y1, t.x2, t.y2) != 0.0f;
            // a pixel centre of the tile inside the closed box exists only if the ranges overlap
            touches = has_area && t.a > 0.0f && !(t.xmax < tile_x0 || t.xmin > tile_x1 || t.ymax < tile_y0 || t.ymin > tile_y1);
        }
        const uint32_t ballot = __ballot_sync(0xffffffffu, touches);
        if (lane == 0) warp_count[warp] = __popc(ballot);
        __syncthreads();
        uint32_t offset = n_keep;
        for (uint32_t w = 0; w < warp; ++w) offset += warp_count[w];
        if (touches) keep[offset + __popc(ballot & ((1u << lane) - 1u))] = static_cast<uint16_t>(k);
        __syncthreads();
        if (tid == 0) {
            uint32_t total = 0;
            for (uint32_t w = 0; w < kPaintThreads / 32; ++w) total += warp_count[w];
            n_keep += total;
        }
        __syncthreads();
    }
    const uint32_t n_list = n_keep;

    // ---- pixel loop: 4 adjacent pixels of one row per thread -------------------------------------
    const uint32_t row = j0 + tid / (kPaintTileW / 4), col = i0 + (tid % (kPaintTileW / 4)) * 4u;
    const float py = __fmul_rn(__fadd_rn(static_cast<float>(row), 0.5f), inv_h);
    float px[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) px[q] = __fmul_rn(__fadd_rn(static_cast<float>(col + q), 0.5f), inv_w);
    float cr[4], cg[4], cb[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) { cr[q] = a.background; cg[q] = a.background; cb[q] = a.background; }

    for (uint32_t n = 0; n < n_list; ++n) {
        const float4* rec = reinterpret_cast<const float4*>(&tri[keep[n]]);
        const float4 va = rec[0], vb = rec[1], vc = rec[2], vd = rec[3];
        const float x0 = va.x, y0 = va.y, x1 = va.z, y1 = va.w, x2 = vb.x, y2 = vb.y;
        const float r = vb.z, g = vb.w, b = vc.x, alpha = vc.y;
        const float xmin = vc.z, xmax = vc.w, ymin = vd.x, ymax = vd.y;
        if (py < ymin || py > ymax) continue;                        // whole thread outside the box
        // the three edges: differences of the vertices once, of the point per pixel
        const float dx0 = __fsub_rn(x1, x0), dy0 = __fsub_rn(y1, y0);
        const float dx1 = __fsub_rn(x2, x1), dy1 = __fsub_rn(y2, y1);
        const float dx2 = __fsub_rn(x0, x2), dy2 = __fsub_rn(y0, y2);
        const float t10 = __fmul_rn(dx0, __fsub_rn(py, y0));
        const float t11 = __fmul_rn(dx1, __fsub_rn(py, y1));
        const float t12 = __fmul_rn(dx2, __fsub_rn(py, y2));
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float e0 = __fsub_rn(t10, __fmul_rn(dy0, __fsub_rn(px[q], x0)));
            const float e1 = __fsub_rn(t11, __fmul_rn(dy1, __fsub_rn(px[q], x1)));
            const float e2 = __fsub_rn(t12, __fmul_rn(dy2, __fsub_rn(px[q], x2)));
            const bool same_sign = (e0 >= 0.0f && e1 >= 0.0f && e2 >= 0.0f) || (e0 <= 0.0f && e1 <= 0.0f && e2 <= 0.0f);
            if (same_sign && px[q] >= xmin && px[q] <= xmax) {
                cr[q] = fmaf(alpha, r - cr[q], cr[q]);
                cg[q] = fmaf(alpha, g - cg[q], cg[q]);
                cb[q] = fmaf(alpha, b - cb[q], cb[q]);
            }
        }
    }

    // ---- squared distance to the target, fixed-order block sum --------------------------------------
    float sq = 0.f;
    if (row < a.H) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (col + q < a.W) {
                const size_t at = (static_cast<size_t>(row) * a.W + col + q) * 3u;
                const float d0 = cr[q] - __ldg(a.target + at), d1 = cg[q] - __ldg(a.target + at + 1), d2 = cb[q] - __ldg(a.target + at + 2);
                sq += d0 * d0 + d1 * d1 + d2 * d2;
                if (a.canvas) {
                    float* out = a.canvas + static_cast<size_t>(member) * a.W * a.H * 3u + at;
                    out[0] = cr[q]; out[1] = cg[q]; out[2] = cb[q];
                }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
    if (lane == 0) warp_sum[warp] = sq;
    __syncthreads();
    if (tid == 0) {
        float total = 0.f;
        for (int w = 0; w < kPaintThreads / 32; ++w) total += warp_sum[w];
        a.partial[static_cast<size_t>(member) * gridDim.y + tile] = total;
    }
}

__global__ void k_paint_finalize(const float* __restrict__ partial, uint32_t P, uint32_t tiles, float inv_count,
                                 float* __restrict__ fitness)
{
    const uint32_t m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= P) return;
    float s = 0.f;
    for (uint32_t t = 0; t < tiles; ++t) s += partial[static_cast<size_t>(m) * tiles + t];
    fitness[m] = -s * inv_count;
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static uint32_t paint_tiles(uint32_t W, uint32_t H)
{
    return ((W + kPaintTileW - 1) / kPaintTileW) * ((H + kPaintTileH - 1) / kPaintTileH);
}

bool paint_supported(uint32_t param_dim, uint32_t W, uint32_t H)
{
    return param_dim % 10u == 0 && param_dim / 10u >= 1 && param_dim / 10u <= kPaintMaxTriangles &&
           W >= 1 && H >= 1 && W <= 4096 && H <= 4096 && paint_tiles(W, H) <= 65535u;
}

size_t paint_scratch_bytes(uint32_t P, uint32_t W, uint32_t H)
{
    return static_cast<size_t>(P) * paint_tiles(W, H) * sizeof(float);
}

int launch_rollout_paint(cudaStream_t st, const float* theta, uint32_t ldD, uint32_t P, uint32_t param_dim,
                         uint32_t W, uint32_t H, float background, const float* target, void* scratch,
                         float* fitness, float* canvas)
{
    PaintArgs a;
    a.theta = theta; a.ldD = ldD; a.P = P; a.n_tri = param_dim / 10u; a.W = W; a.H = H;
    a.background = background; a.target = target; a.partial = static_cast<float*>(scratch); a.canvas = canvas;
    a.tiles_x = (W + kPaintTileW - 1) / kPaintTileW; a.tiles_y = (H + kPaintTileH - 1) / kPaintTileH;
    const uint32_t tiles = a.tiles_x * a.tiles_y;
    dim3 grid(P, tiles);
    const size_t smem = (sizeof(PaintTri) + sizeof(uint16_t)) * a.n_tri;       // at most 33 KB
    k_paint<<<grid, kPaintThreads, smem, st>>>(a);
    if (cudaGetLastError() != cudaSuccess) return -1;
    const float inv = 1.0f / (3.0f * static_cast<float>(W) * static_cast<float>(H));
    k_paint_finalize<<<(P + 255u) / 256u, 256, 0, st>>>(a.partial, P, tiles, inv, fitness);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 2;
}

}  // namespace evo
