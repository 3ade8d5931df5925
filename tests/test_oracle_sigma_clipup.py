"""Pins for the oracle's per-dimension sigma, PGPE sigma update and ClipUp."""
import math

import numpy as np

import oracle


def test_ask_sigma_reduces_to_scalar_ask_and_scales_per_dimension():
    P, D = 8, 37
    c = np.random.default_rng(0).standard_normal(D).astype(np.float32)
    th0, eps0 = oracle.ask(3, 2, P, D, c, 0.25)
    th1, eps1 = oracle.ask_sigma(3, 2, P, D, c, np.full(D, 0.25, np.float32))
    assert (th0.view(np.uint32) == th1.view(np.uint32)).all() and (eps0 == eps1).all()
    sg = np.linspace(0.01, 2.0, D).astype(np.float32)          # powers of two not needed: fma pin below
    th, eps = oracle.ask_sigma(3, 2, P, D, np.zeros(D, np.float32), sg)
    assert (th[0::2] == sg[None, :] * eps).all() and (th[1::2] == -(sg[None, :] * eps)).all()


def test_centre_gradient_with_sigma_vector_matches_brute_force_from_theta():
    P, D = 16, 9
    sg = (2.0 ** np.arange(-4, 5)).astype(np.float32)           # exact products
    th, eps = oracle.ask_sigma(5, 0, P, D, np.zeros(D, np.float32), sg)
    f = np.random.default_rng(1).standard_normal(P).astype(np.float32)
    _, u, _ = oracle.centered_rank(f)
    g = oracle.gradient_sigma(u, eps, sg)
    brute = (u.astype(np.float64)[:, None] * th.astype(np.float64)).sum(0) / P
    assert np.abs(g - brute).max() < 1e-12
    # scalar special case
    assert np.abs(oracle.gradient_sigma(u, eps, np.full(D, 0.5)) - oracle.gradient(u, eps, 0.5)).max() < 1e-15


def test_sigma_gradient_matches_the_definition_on_perturbations():
    # written from theta alone: e = theta+ - centre, S = sum_j ((u+ + u-)/2 - b)(e^2 - sigma^2)/sigma / H
    P, D = 4, 3
    sg = np.array([0.5, 0.25, 2.0], dtype=np.float32)
    c = np.zeros(D, np.float32)
    th, eps = oracle.ask_sigma(9, 1, P, D, c, sg)
    f = np.array([0.3, -1.0, 2.0, 0.1], dtype=np.float32)
    _, u, _ = oracle.centered_rank(f)
    gs = oracle.sigma_gradient(u, eps, sg)
    b = float(u.astype(np.float64).mean())
    brute = np.zeros(D)
    for d in range(D):
        for j in range(P // 2):
            e = float(th[2 * j, d])
            s = 0.5 * (float(u[2 * j]) + float(u[2 * j + 1])) - b
            brute[d] += s * (e * e - float(sg[d]) ** 2) / float(sg[d])
        brute[d] /= (P // 2)
    assert np.abs(gs - brute).max() < 1e-12


def test_sigma_gradient_scale_on_a_quadratic_fitness():
    """Pins the SCALE (the power of sigma) of the PGPE sigma gradient against mathematics.

    Feed un-ranked weights u_m = f(theta_m) with f(theta) = sum_d a_d theta_d^2, centre 0 and a
    different sigma in every dimension.  Both members of an antithetic pair then score the same,
    s_j = f(theta_j+) = sum_k a_k sigma_k^2 eps_jk^2, and the baseline is b = mean(u) ~ E f.  The
    symmetric-sampling estimate is gs_d = mean_j (s_j - b) (e_jd^2 - sigma_d^2) / sigma_d with
    e = sigma_d eps, hence
        E[gs_d] = Cov(f, e_d^2) / sigma_d = a_d Var(e_d^2) / sigma_d = a_d (2 sigma_d^4) / sigma_d
                = 2 a_d sigma_d^3
    (Var of sigma^2 chi^2_1 is 2 sigma^4; the other dimensions are independent of e_d).  That is
    sigma_d^2 times the exact derivative d/d sigma_d E[f] = 2 a_d sigma_d, as it must be for
    Sehnke's (e^2 - sigma^2)/sigma, which is the likelihood-ratio term times sigma^2.  A slip of
    one power of sigma (dividing by sigma^2, or not at all) is off by factors of 0.3 .. 2 here.
    Standard error with H = 2e5 pairs: below 1 % per dimension; the bound is 5 %."""
    H, D = 200_000, 4
    sg = np.array([0.3, 0.7, 1.3, 2.0])
    a = np.array([1.5, -0.8, 0.25, 0.1])
    th, eps = oracle.ask_sigma(21, 0, 2 * H, D, np.zeros(D, np.float32), sg.astype(np.float32))
    u = (a[None, :] * th.astype(np.float64) ** 2).sum(1).astype(np.float32)
    gs = oracle.sigma_gradient(u, eps, sg.astype(np.float32).astype(np.float64))
    want = 2.0 * a * sg ** 3
    assert np.all(np.abs(gs - want) < 0.05 * np.abs(want)), (gs, want)
    # the neighbouring wrong scalings are far outside the bound
    assert np.any(np.abs(gs - want / sg) > 0.2 * np.abs(want)) and np.any(np.abs(gs - want * sg) > 0.2 * np.abs(want))


def test_sigma_gradient_sign_and_zero_cases():
    P, D = 512, 6
    sg = np.full(D, 0.3)
    _, eps = oracle.ask_sigma(11, 0, P, D, np.zeros(D, np.float32), sg.astype(np.float32))
    # fitness rewards large perturbations in dimension 0, small ones in dimension 1
    e = eps.astype(np.float64)
    pair_score = e[:, 0] ** 2 - e[:, 1] ** 2
    f = np.repeat(pair_score, 2).astype(np.float32)              # both members of a pair share it
    _, u, _ = oracle.centered_rank(f)
    gs = oracle.sigma_gradient(u, eps, sg)
    assert gs[0] > 0 and gs[1] < 0
    assert np.abs(gs[2:]).max() < 0.3 * max(gs[0], -gs[1])
    # if only the SIGN of the perturbation matters (antisymmetric fitness), pairs carry no sigma signal
    f2 = np.empty(P, np.float32); f2[0::2] = e[:, 0]; f2[1::2] = -e[:, 0]
    _, u2, _ = oracle.centered_rank(f2)
    s_pair = 0.5 * (u2[0::2].astype(np.float64) + u2[1::2])
    assert np.abs(s_pair).max() < 2.0 / P
    assert np.abs(oracle.sigma_gradient(u2, eps, sg)).max() < 2e-3


def test_sigma_update_step_and_clip():
    sg = np.array([1.0, 1.0, 1.0, 0.5])
    gs = np.array([0.5, 10.0, -10.0, -0.2])
    new = oracle.sigma_update(sg, gs, 0.1, 0.2)
    assert np.allclose(new, [1.05, 1.2, 0.8, 0.48], atol=1e-15)
    assert (new > 0).all()


def test_clipup_normalised_step_momentum_and_clip():
    g = np.array([3.0, 4.0])
    c, v = oracle.clipup(np.zeros(2), np.zeros(2), g, lr=0.1, momentum=0.9, max_speed=0.15)
    assert np.allclose(v, [0.06, 0.08]) and np.allclose(c, v)              # |v| = lr
    c, v = oracle.clipup(c, v, g, 0.1, 0.9, 0.15)                          # 0.9*0.1 + 0.1 = 0.19 -> clipped
    assert abs(np.linalg.norm(v) - 0.15) < 1e-15 and np.allclose(v / np.linalg.norm(v), [0.6, 0.8])
    assert np.allclose(c, np.array([0.06, 0.08]) + v)
    # scale invariance in g, and a zero gradient leaves only the momentum term
    c1, v1 = oracle.clipup(np.zeros(2), np.zeros(2), 1000 * g, 0.1, 0.9, 1.0)
    assert np.allclose(v1, [0.06, 0.08])
    c2, v2 = oracle.clipup(np.zeros(2), np.array([0.1, 0.0]), np.zeros(2), 0.1, 0.9, 1.0)
    assert np.allclose(v2, [0.09, 0.0]) and np.allclose(c2, v2)
