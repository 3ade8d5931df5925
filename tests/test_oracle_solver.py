"""Pins for the oracle's ask/tell: identities, brute force, and a library optimiser."""
import numpy as np
import torch

import oracle


def test_ask_antithetic_pairs():
    P, D = 16, 385
    center = np.zeros(D, dtype=np.float32)
    theta, eps = oracle.ask(0, 0, P, D, center, 0.1)
    # centre 0: theta+ = -theta- exactly, so pairs sum to 2*centre = 0
    assert (theta[0::2] + theta[1::2] == 0).all()
    # the + member is the even one
    assert (theta[0::2] == (np.float32(0.1) * eps)).all()
    rng = np.random.default_rng(0)
    center = rng.standard_normal(D).astype(np.float32)
    theta, eps = oracle.ask(5, 9, P, D, center, 0.1)
    resid = np.abs(theta[0::2].astype(np.float64) + theta[1::2] - 2.0 * center)
    bound = 2.0**-23 * (np.abs(center) + np.abs(0.1 * eps.astype(np.float64))) + 1e-30
    assert (resid <= bound).all()
    # each entry is the single-rounding fma of the definition
    want = (np.float64(np.float32(0.1)) * eps[3].astype(np.float64) + center).astype(np.float32)
    assert (theta[6] == want).all()
    # rows of eps are the per-pair noise rows
    assert (eps[5] == oracle.eps_row(5, 9, 5, D)).all()


def test_rank_is_permutation_and_matches_sort():
    rng = np.random.default_rng(1)
    for P in (2, 16, 256, 1001 * 2):
        f = rng.standard_normal(P).astype(np.float32)
        rank, u, bad = oracle.centered_rank(f)
        assert not bad
        assert sorted(rank.tolist()) == list(range(P))
        order = np.argsort(f, kind="stable")
        want = np.empty(P, dtype=np.int32); want[order] = np.arange(P)
        assert (rank == want).all()
        assert u.min() == -0.5 and u.max() == 0.5
        assert abs(float(u.astype(np.float64).sum())) < 1e-4
        assert (u == (rank.astype(np.float32) / np.float32(P - 1) - np.float32(0.5))).all()


def test_rank_ties_and_specials():
    f = np.array([1.0, 1.0, 1.0, 1.0], dtype=np.float32)
    rank, u, bad = oracle.centered_rank(f)
    assert rank.tolist() == [0, 1, 2, 3]
    f = np.array([0.0, -0.0, np.inf, -np.inf, 2.0, 2.0], dtype=np.float32)
    rank, _, bad = oracle.centered_rank(f)
    assert not bad and rank.tolist() == [1, 2, 5, 0, 3, 4]
    _, _, bad = oracle.centered_rank(np.array([0.0, np.nan], dtype=np.float32))
    assert bad


def test_gradient_matches_brute_force_from_theta_alone():
    # sigma a power of two and centre 0, so theta = +-sigma*eps exactly and the
    # population-form estimator g = (1/P) sum_m u_m (theta_m - centre) uses theta only
    P, D, sigma = 4, 3, 0.5
    theta, eps = oracle.ask(11, 0, P, D, np.zeros(D, dtype=np.float32), sigma)
    f = np.array([0.3, -1.0, 2.0, 0.1], dtype=np.float32)
    _, u, _ = oracle.centered_rank(f)
    g = oracle.gradient(u, eps, sigma)
    brute = np.zeros(D)
    for d in range(D):
        for m in range(P):
            brute[d] += float(u[m]) * float(theta[m, d])
        brute[d] /= P
    assert np.abs(g - brute).max() < 1e-12
    # larger random case, same identity
    P, D = 64, 50
    theta, eps = oracle.ask(12, 1, P, D, np.zeros(D, dtype=np.float32), sigma)
    f = np.random.default_rng(2).standard_normal(P).astype(np.float32)
    _, u, _ = oracle.centered_rank(f)
    g = oracle.gradient(u, eps, sigma)
    brute = (u.astype(np.float64)[:, None] * theta.astype(np.float64)).sum(0) / P
    assert np.abs(g - brute).max() < 1e-12


def test_gradient_points_uphill_on_a_linear_fitness():
    # fitness = a . theta: the estimate must correlate positively with a
    P, D, sigma = 512, 20, 0.1
    a = np.random.default_rng(3).standard_normal(D)
    theta, eps = oracle.ask(13, 0, P, D, np.zeros(D, dtype=np.float32), sigma)
    f = (theta.astype(np.float64) @ a).astype(np.float32)
    _, u, _ = oracle.centered_rank(f)
    g = oracle.gradient(u, eps, sigma)
    cos = float(g @ a / np.linalg.norm(g) / np.linalg.norm(a))
    assert cos > 0.8


def test_adam_matches_torch_maximize():
    rng = np.random.default_rng(4)
    D, lr = 37, 0.01
    c0 = rng.standard_normal(D)
    p = torch.tensor(c0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=lr, betas=(0.9, 0.999), eps=1e-8, maximize=True)
    c, m, v = c0.copy(), np.zeros(D), np.zeros(D)
    for t in range(1, 8):
        g = rng.standard_normal(D) * 10.0 ** rng.integers(-3, 2)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        c, m, v = oracle.adam(c, m, v, g, t, lr)
        assert np.abs(c - p.detach().numpy()).max() < 1e-13


def test_adam_first_step_is_lr_times_sign():
    g = np.array([3.0, -2e-3, 1e-5, -7.0])
    c, m, v = oracle.adam(np.zeros(4), np.zeros(4), np.zeros(4), g, 1, 0.01)
    want = 0.01 * g / (np.abs(g) + 1e-8)
    assert np.abs(c - want).max() < 1e-15
    # |step| = lr / (1 + eps/|g|): within eps/|g| of lr
    assert (np.abs(np.abs(c) - 0.01) <= 0.01 * 1e-8 / np.abs(g) * 1.001).all()
    # constant gradient: the step tends to lr
    c, m, v = np.zeros(1), np.zeros(1), np.zeros(1)
    for t in range(1, 200):
        prev = c.copy()
        c, m, v = oracle.adam(c, m, v, np.array([0.37]), t, 0.01)
    assert abs((c - prev)[0] - 0.01) < 1e-8
