/*
 * CPU oracle (test infrastructure only): the triangle-painting task (paper Section 3, "Concrete and
 * Abstract Painting": a canvas painted with semi-transparent triangles is fitted to a target image by
 * an evolution strategy that is used on its own, the task being the caller's).
 *
 * The paper gives no detail of the task; the conventions below are this repository's readings.
 * A member is N triangles of 10 numbers each: x0 y0 x1 y1 x2 y2 r g b a.  Every number v is mapped
 * to the unit interval by u = min(max(0.5 + 0.5 v, 0), 1).  The canvas is the unit square sampled at
 * pixel centres ((i + 0.5) / W, (j + 0.5) / H), it starts at the grey level `background`, and the
 * triangles are composited in order: where pixel p is inside triangle k, C <- C + a_k (c_k - C).
 * Fitness = -mean over pixels and channels of (C - target)^2.
 *
 * Which pixels a triangle covers is an integer decision, so it is DEFINED in fp32, each step a
 * single correctly rounded operation: u = fmaf(0.5f, v, 0.5f) clamped; for an edge from a to b,
 * e(p) = (bx - ax) * (py - ay) - (by - ay) * (px - ax) with the two differences, the two products
 * and the final difference each rounded once; p is inside when it lies in the closed bounding box of
 * the three vertices and the three edge values are all >= 0 or all <= 0; a triangle whose own third
 * vertex has edge value 0 (no area) paints nothing.  (The bounding box keeps a needle-thin triangle,
 * whose three edge lines nearly coincide, from claiming pixels far beyond its tips through rounding.)
 * Colours and compositing are plain real arithmetic (fp64 here).
 */
#include "oracle.h"

#include <math.h>

static float unit_f32(float v)
{
    float u = fmaf(0.5f, v, 0.5f);
    if (!(u >= 0.0f)) u = 0.0f;             /* NaN -> 0 as well */
    if (u > 1.0f) u = 1.0f;
    return u;
}

/* fp32 edge value of point (px, py) against the edge a -> b, every operation rounded once
 * (the file is compiled without contraction) */
static float edge_f32(float ax, float ay, float bx, float by, float px, float py)
{
    const float dx = bx - ax, dy = by - ay;
    const float qx = px - ax, qy = py - ay;
    const float t1 = dx * qy;
    const float t2 = dy * qx;
    return t1 - t2;
}

int oracle_paint_inside(const float tri[6], float px, float py)
{
    const float x0 = unit_f32(tri[0]), y0 = unit_f32(tri[1]);
    const float x1 = unit_f32(tri[2]), y1 = unit_f32(tri[3]);
    const float x2 = unit_f32(tri[4]), y2 = unit_f32(tri[5]);
    if (edge_f32(x0, y0, x1, y1, x2, y2) == 0.0f) return 0;
    if (px < fminf(x0, fminf(x1, x2)) || px > fmaxf(x0, fmaxf(x1, x2))) return 0;
    if (py < fminf(y0, fminf(y1, y2)) || py > fmaxf(y0, fmaxf(y1, y2))) return 0;
    const float e0 = edge_f32(x0, y0, x1, y1, px, py);
    const float e1 = edge_f32(x1, y1, x2, y2, px, py);
    const float e2 = edge_f32(x2, y2, x0, y0, px, py);
    return (e0 >= 0.0f && e1 >= 0.0f && e2 >= 0.0f) || (e0 <= 0.0f && e1 <= 0.0f && e2 <= 0.0f);
}

void oracle_paint_render(const float* params, uint32_t n_triangles, uint32_t W, uint32_t H,
                         double background, double* canvas)
{
    const float inv_w = 1.0f / (float)W, inv_h = 1.0f / (float)H;
    for (uint32_t j = 0; j < H; ++j)
        for (uint32_t i = 0; i < W; ++i) {
            const float px = ((float)i + 0.5f) * inv_w;
            const float py = ((float)j + 0.5f) * inv_h;
            double c[3] = { background, background, background };
            for (uint32_t k = 0; k < n_triangles; ++k) {
                const float* t = params + (size_t)k * 10;
                if (!oracle_paint_inside(t, px, py)) continue;
                const double a = (double)unit_f32(t[9]);
                for (int ch = 0; ch < 3; ++ch)
                    c[ch] = c[ch] + a * ((double)unit_f32(t[6 + ch]) - c[ch]);
            }
            for (int ch = 0; ch < 3; ++ch) canvas[((size_t)j * W + i) * 3 + ch] = c[ch];
        }
}

double oracle_paint_fitness(const float* params, uint32_t n_triangles, uint32_t W, uint32_t H,
                            double background, const float* target, double* canvas)
{
    oracle_paint_render(params, n_triangles, W, H, background, canvas);
    double s = 0.0;
    const size_t n = (size_t)W * H * 3;
    for (size_t i = 0; i < n; ++i) {
        const double d = canvas[i] - (double)target[i];
        s += d * d;
    }
    return -s / (double)n;
}
