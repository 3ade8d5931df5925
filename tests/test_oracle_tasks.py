"""Pins for the oracle's tasks: conservation laws, equilibria, closed forms, hand cases."""
import math

import numpy as np

import oracle

PI32 = float(np.float32(math.pi))


def test_cartpole_energy_and_momentum_conserved_without_force():
    p = oracle.cartpole_params()
    rng = np.random.default_rng(0)
    for a in (0.05, 0.2):
        for _ in range(10):
            s = np.array([0, 0, math.pi, 0]) + rng.uniform(-a, a, 4)
            e0, m0 = oracle.cartpole_energy(p, s), oracle.cartpole_momentum(p, s)
            for _ in range(100):
                s = oracle.cartpole_step(p, s, 0.0)
            assert abs(oracle.cartpole_energy(p, s) - e0) < 1e-9
            assert abs(oracle.cartpole_momentum(p, s) - m0) < 1e-10


def test_cartpole_euler_variant_is_first_order():
    p = oracle.cartpole_params(integrator=1)
    s = np.array([0.0, 0.0, math.pi + 0.2, 0.1])
    e0 = oracle.cartpole_energy(p, s)
    for _ in range(100):
        s = oracle.cartpole_step(p, s, 0.0)
    assert 1e-6 < abs(oracle.cartpole_energy(p, s) - e0) < 1e-1


def test_cartpole_equilibria_and_force_direction():
    p = oracle.cartpole_params()
    for theta in (0.0, math.pi):
        s = np.array([0.3, 0.0, theta, 0.0])
        for _ in range(50):
            s = oracle.cartpole_step(p, s, 0.0)
        assert abs(s[0] - 0.3) < 1e-12 and abs(s[1]) < 1e-12 and abs(s[3]) < 1e-12 \
            and abs(s[2] - theta) < 1e-12
    # a push to the right accelerates the cart to the right
    s = oracle.cartpole_step(p, np.array([0, 0, math.pi, 0.0]), 10.0)
    assert s[1] > 0 and s[0] > 0
    # upright pole with a small tilt falls further
    s = np.array([0, 0, 0.01, 0.0])
    for _ in range(20):
        s = oracle.cartpole_step(p, s, 0.0)
    assert s[2] > 0.01


def test_cartpole_small_angle_period_about_the_bottom():
    p = oracle.cartpole_params()
    period = 2 * math.pi * math.sqrt((4.0 / 3.0 - 0.1 / 1.1) * 0.5 / 9.8)
    s = np.array([0.0, 0.0, math.pi + 1e-4, 0.0])
    # momentum is zero; find the time of the second downward zero crossing of (theta - pi)
    prev, t_cross, n = s[2] - math.pi, [], 0
    for i in range(1, 400):
        s = oracle.cartpole_step(p, s, 0.0)
        cur = s[2] - math.pi
        if prev > 0 >= cur or prev < 0 <= cur:
            t_cross.append((i - 1 + prev / (prev - cur)) * p.dt)
        prev = cur
    assert len(t_cross) >= 3
    assert abs((t_cross[2] - t_cross[0]) - period) < 2e-4 * period


def test_cartpole_reset_is_seeded_uniform_about_pole_down():
    a = 0.2
    s = np.stack([oracle.cartpole_reset(0, g, e, a) for g in range(20) for e in range(50)])
    d = s - np.array([0, 0, PI32, 0], dtype=np.float32)
    assert (np.abs(d) <= a * (1 + 1e-6)).all()
    assert abs(d.mean()) < 0.02 and abs(d.std() - a / math.sqrt(3)) < 0.01
    r = oracle.stream_words(0, 1, 3, 7, 0)
    want = [np.float32(2 * a) * np.float32(oracle.u_half(int(x))) for x in r]
    got = oracle.cartpole_reset(0, 3, 7, a)
    assert abs(float(got[0]) - (float(want[0]) - a)) < 1e-7


def test_cartpole_zero_policy_is_the_free_pendulum_and_reward_is_bounded():
    p = oracle.cartpole_params()
    sizes = [5, 16, 16, 1]
    theta = np.zeros(385, dtype=np.float32)
    E, T = 2, 150
    fit, trace = oracle.rollout_cartpole(theta, sizes, 10.0, p, 0.05, 0, 0, E, T, want_trace=True)
    total = 0.0
    for e in range(E):
        s = oracle.cartpole_reset(0, 0, e, 0.05).astype(np.float64)
        for t in range(T):
            s = oracle.cartpole_step(p, s, 0.0)
            total += math.cos(s[2]) * math.exp(-s[0] ** 2)
            assert np.abs(trace[e, t] - s).max() < 1e-13
    assert abs(fit - total / E) < 1e-12
    assert abs(fit) <= T
    # a random policy still respects |return| <= T
    rng = np.random.default_rng(1)
    fit, _ = oracle.rollout_cartpole(rng.standard_normal(385).astype(np.float32), sizes, 10.0, p,
                                     0.05, 0, 0, 1, 200)
    assert abs(fit) <= 200


def test_cartpole_rollout_uses_policy_force_and_observation_order():
    # 5 -> 1 policy reading only observation slot 4 (theta_dot) with a small gain
    p = oracle.cartpole_params()
    sizes = [5, 1]
    theta = np.zeros(6, dtype=np.float32); theta[4] = 0.5
    fit, trace = oracle.rollout_cartpole(theta, sizes, 10.0, p, 0.05, 3, 2, 1, 5, want_trace=True)
    s = oracle.cartpole_reset(3, 2, 0, 0.05).astype(np.float64)
    ret = 0.0
    for t in range(5):
        force = 10.0 * math.tanh(0.5 * s[3])
        s = oracle.cartpole_step(p, s, force)
        ret += math.cos(s[2]) * math.exp(-s[0] ** 2)
        assert np.abs(trace[0, t] - s).max() < 1e-13
    assert abs(fit - ret) < 1e-13
    # slot 2 is cos(theta), slot 3 is sin(theta)
    for slot, fn in ((2, math.cos), (3, math.sin)):
        theta = np.zeros(6, dtype=np.float32); theta[slot] = 1.0
        _, trace = oracle.rollout_cartpole(theta, sizes, 10.0, p, 0.05, 3, 2, 1, 1, want_trace=True)
        s = oracle.cartpole_reset(3, 2, 0, 0.05).astype(np.float64)
        s = oracle.cartpole_step(p, s, 10.0 * math.tanh(fn(s[2])))
        assert np.abs(trace[0, 0] - s).max() < 1e-13


def test_tanh_linear_constants_scale_and_layout():
    A, B = oracle.tanh_linear_constants(2)
    assert A.shape == (28, 28) and B.shape == (28, 8)
    assert abs(A.std() - 0.9 / math.sqrt(28)) < 0.02 and abs(B.std() - 1 / math.sqrt(8)) < 0.04
    z = oracle.normal4(oracle.stream_words(2, 4, 0, 0, 5))
    assert (A.reshape(-1)[20:24] == z * np.float32(0.9 / math.sqrt(28))).all()
    z = oracle.normal4(oracle.stream_words(2, 4, 0, 1, 5))
    assert (B.reshape(-1)[20:24] == z * np.float32(1 / math.sqrt(8))).all()


def test_tanh_linear_zero_policy_recurrence_by_hand():
    A, B = oracle.tanh_linear_constants(2)
    sizes = [28, 128, 128, 8]
    theta = np.zeros(21256, dtype=np.float32)
    fit, trace = oracle.rollout_tanh_linear(theta, sizes, 1.0, A, B, 2, 1, 2, 3, want_trace=True)
    total = 0.0
    for e in range(2):
        x = oracle.tanh_linear_reset(2, 1, e).astype(np.float64)
        for t in range(3):
            total += -(x @ x)
            x = np.tanh(A.astype(np.float64) @ x)
            assert np.abs(trace[e, t] - x).max() < 1e-14
    assert abs(fit - total / 2) < 1e-12


def test_tanh_linear_uses_actions_and_reward_bounds():
    A, B = oracle.tanh_linear_constants(2)
    sizes = [28, 8]                    # one layer: a = tanh(W x + b)
    rng = np.random.default_rng(5)
    theta = (rng.standard_normal(28 * 8 + 8) * 0.3).astype(np.float32)
    W = theta[:224].reshape(8, 28).astype(np.float64); b = theta[224:].astype(np.float64)
    T = 6
    fit, trace = oracle.rollout_tanh_linear(theta, sizes, 1.0, A, B, 2, 0, 1, T, want_trace=True)
    x = oracle.tanh_linear_reset(2, 0, 0).astype(np.float64)
    ret = 0.0
    for t in range(T):
        a = np.tanh(W @ x + b)
        r = -(x @ x) - 0.01 * (a @ a)
        if t >= 1:
            assert -28.08 <= r <= 0.0
        ret += r
        x = np.tanh(A.astype(np.float64) @ x + B.astype(np.float64) @ a)
        assert np.abs(trace[0, t] - x).max() < 1e-14
    assert abs(fit - ret) < 1e-12
