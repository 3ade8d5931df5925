"""Pins of the triangle-painting oracle (paper Section 3, "Concrete and Abstract Painting"): coverage
counted by hand, blending in closed form, invariances, and an independent barycentric rasteriser."""
import itertools

import numpy as np

import oracle


def raw(u):
    """Raw parameter whose unit-interval image is u (u = 0.5 + 0.5 v)."""
    return 2.0 * np.asarray(u, dtype=np.float64) - 1.0


def tri(p0, p1, p2, rgb, a):
    return np.array([*raw(p0), *raw(p1), *raw(p2), *raw(rgb), float(raw(a))], np.float32)


def test_right_triangle_covers_the_hand_counted_pixels_edges_included():
    # x + y <= 1 on an 8x8 canvas: centres ((i+.5)/8, (j+.5)/8) with i + j <= 7 -> 36 pixels,
    # the 8 pixels with i + j = 7 lie exactly on the hypotenuse and count as inside
    c = oracle.paint_render(tri((0, 0), (1, 0), (0, 1), (1, 1, 1), 1.0)[None], 8, 8)
    want = np.add.outer(np.arange(8), np.arange(8)) <= 7
    assert np.array_equal(c[:, :, 0] == 1.0, want) and c.sum() == 3 * 36


def test_axis_aligned_half_plane_and_row_column_orientation():
    # left half (x <= 0.5) as two triangles; canvas index order is [row = y][column = x]
    p = np.stack([tri((0, 0), (0.5, 0), (0.5, 1), (1, 0, 0), 1.0), tri((0, 0), (0.5, 1), (0, 1), (1, 0, 0), 1.0)])
    c = oracle.paint_render(p, 16, 4)
    assert c.shape == (4, 16, 3)
    assert np.all(c[:, :8, 0] == 1.0) and np.all(c[:, 8:, 0] == 0.0) and np.all(c[:, :, 1:] == 0.0)


def test_blending_order_and_background_in_closed_form():
    full = [((0, 0), (1, 0), (0, 1)), ((1, 1), (1, 0), (0, 1))]          # two halves of the square
    def layer(rgb, a):
        return [tri(*f, rgb, a) for f in full]
    p = np.stack(layer((1.0, 0.0, 0.5), 0.25) + layer((0.0, 1.0, 0.5), 0.5))
    c = oracle.paint_render(p, 6, 6, background=0.2)
    # interior pixels are covered once per layer; the diagonal pixels belong to both halves
    inner = np.add.outer(np.arange(6), np.arange(6)) != 5
    first = 0.2 + 0.25 * (np.array([1.0, 0.0, 0.5]) - 0.2)
    want = first + 0.5 * (np.array([0.0, 1.0, 0.5]) - first)
    assert np.allclose(c[inner], want, atol=1e-7)                         # unit_f32 of 0.25 etc. is exact
    swapped = oracle.paint_render(p[[2, 3, 0, 1]], 6, 6, background=0.2)
    assert not np.allclose(swapped[inner], want, atol=1e-3)               # compositing is ordered


def test_vertex_order_and_orientation_do_not_matter():
    rng = np.random.default_rng(3)
    p = rng.standard_normal((6, 10)).astype(np.float32)
    ref = oracle.paint_render(p, 32, 24)
    for perm in itertools.permutations(range(3)):
        q = p.copy()
        q[:, :6] = p[:, :6].reshape(6, 3, 2)[:, list(perm), :].reshape(6, 6)
        assert np.array_equal(oracle.paint_render(q, 32, 24), ref)


def test_degenerate_and_transparent_triangles_paint_nothing_and_parameters_clamp():
    bg = 0.3
    p = np.stack([tri((0.2, 0.2), (0.2, 0.2), (0.2, 0.2), (1, 1, 1), 1.0),        # a point
                  tri((0.1, 0.1), (0.5, 0.5), (0.9, 0.9), (1, 1, 1), 1.0),        # a segment through pixel centres
                  tri((0, 0), (1, 0), (0, 1), (1, 1, 1), 0.0)])                   # transparent
    assert np.all(oracle.paint_render(p, 10, 10, background=bg) == bg)
    big = np.array([[-9, -9, 9, -9, -9, 9, 7, -7, 0, 5]], np.float32)             # clamps to the unit square
    same = tri((0, 0), (1, 0), (0, 1), (1, 0, 0.5), 1.0)[None]
    assert np.array_equal(oracle.paint_render(big, 12, 12), oracle.paint_render(same, 12, 12))


def _barycentric_cover(t, W, H, margin):
    """Independent rasteriser: barycentric coordinates in fp64 from the solved 2x2 system; returns
    (inside mask, mask of pixels farther than `margin` from every edge in barycentric units)."""
    u = np.clip(0.5 + 0.5 * t[:6].astype(np.float32), 0, 1).astype(np.float64).reshape(3, 2)
    xs = (np.arange(W) + 0.5) / W
    ys = (np.arange(H) + 0.5) / H
    X, Y = np.meshgrid(xs, ys)
    M = np.array([[u[1, 0] - u[0, 0], u[2, 0] - u[0, 0]], [u[1, 1] - u[0, 1], u[2, 1] - u[0, 1]]])
    if abs(np.linalg.det(M)) < 1e-12:
        return np.zeros((H, W), bool), np.zeros((H, W), bool)
    inv = np.linalg.inv(M)
    l1 = inv[0, 0] * (X - u[0, 0]) + inv[0, 1] * (Y - u[0, 1])
    l2 = inv[1, 0] * (X - u[0, 0]) + inv[1, 1] * (Y - u[0, 1])
    l0 = 1 - l1 - l2
    lam = np.stack([l0, l1, l2])
    return np.all(lam >= 0, axis=0), np.all(np.abs(lam) > margin, axis=0)


def test_coverage_matches_a_barycentric_rasteriser_away_from_edges():
    rng = np.random.default_rng(11)
    W, H = 40, 28
    checked = 0
    for _ in range(60):
        t = np.zeros(10, np.float32)
        t[:6] = rng.uniform(-1.2, 1.2, 6)
        t[6:9] = 1.0; t[9] = 1.0                                       # opaque white on black
        c = oracle.paint_render(t[None], W, H)[:, :, 0] == 1.0
        inside, clear = _barycentric_cover(t, W, H, 1e-4)
        assert np.array_equal(c[clear], inside[clear])
        checked += int(clear.sum())
    assert checked > 50000


def test_fitness_is_minus_mean_squared_error_and_zero_on_its_own_rendering():
    rng = np.random.default_rng(5)
    p = rng.standard_normal((12, 10)).astype(np.float32)
    W, H = 20, 16
    canvas = oracle.paint_render(p, W, H, background=0.1)
    target = rng.random((H, W, 3), dtype=np.float32)
    f = oracle.paint_fitness(p, W, H, target, background=0.1)
    assert abs(f + np.mean((canvas - target.astype(np.float64)) ** 2)) < 1e-15
    assert abs(oracle.paint_fitness(p, W, H, canvas.astype(np.float32), background=0.1)) < 1e-14
    assert abs(oracle.paint_fitness(np.zeros((0, 10), np.float32), W, H, target, background=0.1)
               + np.mean((0.1 - target.astype(np.float64)) ** 2)) < 1e-15


def test_single_pixel_inside_decision_is_taken_in_fp32():
    # a point that fp64 puts just outside but whose fp32 edge value rounds to exactly 0 is inside
    t = np.array([*raw((0.1, 0.1)), *raw((0.7, 0.3)), *raw((0.2, 0.9))], np.float32)
    u = np.clip(np.float32(0.5) + np.float32(0.5) * t, 0, 1).astype(np.float32)
    # walk along the first edge: points a + s (b - a) computed in fp32
    hits = 0
    for s in np.linspace(0.05, 0.95, 400, dtype=np.float32):
        px = np.float32(u[0] + s * (u[2] - u[0])); py = np.float32(u[1] + s * (u[3] - u[1]))
        dx, dy = np.float32(u[2] - u[0]), np.float32(u[3] - u[1])
        e = np.float32(np.float32(dx * np.float32(py - u[1])) - np.float32(dy * np.float32(px - u[0])))
        # the oracle's decision must agree with the sign of this fp32 value for the first edge
        inside = oracle.paint_inside(t, px, py)
        area = np.float32(np.float32(dx * np.float32(u[5] - u[1])) - np.float32(dy * np.float32(u[4] - u[0])))
        if (e > 0) != (area > 0) and e != 0:
            assert not inside
            hits += 1
    assert hits > 20


def test_needle_triangle_stays_inside_its_bounding_box():
    # nearly collinear vertices: without the bounding box, rounding could let pixels on the
    # extension of the needle pass the three edge tests
    t = tri((0.30, 0.30), (0.50, 0.50), (0.40, 0.4000001), (1, 1, 1), 1.0)
    c = oracle.paint_render(t[None], 200, 200)[:, :, 0]
    ys, xs = np.nonzero(c)
    if len(xs):
        assert xs.min() >= 0.30 * 200 - 1 and xs.max() <= 0.50 * 200 and ys.min() >= 0.30 * 200 - 1 and ys.max() <= 0.50 * 200
    for px, py in ((0.7, 0.7), (0.1, 0.1), (0.9, 0.9000001)):
        assert not oracle.paint_inside(t[:6], px, py)
