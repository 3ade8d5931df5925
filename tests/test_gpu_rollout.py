"""Control-task rollouts on the GPU against the oracle (teacher-forced: same parameters,
same seeded initial states): per-step state <= 1e-4, fitness <= 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err, oracle_fitness, cartpole_features
from paper_2202_05008_b200 import Solver, workloads as W
from paper_2202_05008_b200.binding import ROLLOUT_GENERIC, ROLLOUT_TILED, ROLLOUT_AUTO, EvoError

pytestmark = pytest.mark.gpu

STATE_TOL, FIT_TOL = 1e-4, 1e-3


def _state_dim(w):
    return 4 if w.task_kind == W.TASK_CARTPOLE else 28


def _rollout_check(w, T, members, kernel, theta_np=None, generation=0, check_trace=True):
    """Roll `members` rows on the GPU (whole population is rolled; rows are compared)."""
    w = w.with_(horizon=T)
    s = Solver(w, trace_steps=T if check_trace else 0, rollout_kernel=kernel)
    if theta_np is None:
        theta_dev = s.ask()
        theta_np = theta_dev.cpu().numpy()
        arg = None
    else:
        arg = s.padded_rows(w.pop_size)
        arg[:, :w.param_dim] = torch.tensor(theta_np, device="cuda")
    sd = _state_dim(w)
    trace = torch.zeros(w.pop_size, w.episodes, T, sd, device="cuda") if check_trace else None
    fit = s.rollout(arg, trace=trace).cpu().numpy()
    assert s.sync_status() == 0
    fit_o, traces_o = oracle_fitness(w, theta_np[members], generation, T, want_trace=check_trace)
    assert rel_err(fit[members], fit_o, floor=1.0) < FIT_TOL
    if check_trace:
        tr = trace.cpu().numpy()
        for k, m in enumerate(members):
            got, want = tr[m].astype(np.float64), traces_o[k]
            if w.task_kind == W.TASK_CARTPOLE:
                got, want = cartpole_features(got), cartpole_features(want)
            for i in range(got.shape[-1]):          # per state component, floor = its RMS
                assert rel_err(got[..., i], want[..., i]) < STATE_TOL, (m, i)
    s.close()
    return fit


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_AUTO])
def test_cfg1_full(kernel):
    fit = _rollout_check(W.CFG1, 200, list(range(16)), kernel)
    assert np.abs(fit).max() <= 200


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_AUTO])
def test_cfg1_random_policies_strong_forces(kernel):
    theta = W.random_parameters(1, 16, 385, scale=0.7)
    _rollout_check(W.CFG1, 200, list(range(16)), kernel, theta_np=theta)


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_AUTO])
def test_cfg2_T200_sampled_members(kernel):
    _rollout_check(W.CFG2, 200, [0, 1, 77, 128, 255], kernel)


# AUTO = the tensor-core kernel (wide layers as split-fp16 tcgen05 MMAs), TILED = the fp32-pipe kernel
@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_TILED, ROLLOUT_AUTO])
def test_cfg4_T200_sampled_members(kernel):
    _rollout_check(W.CFG4, 200, [0, 1, 591, 592, 2047, 4095], kernel)


@pytest.mark.parametrize("pop,episodes", [(2, 4), (6, 3), (10, 6), (1186, 4), (6, 9)])
def test_cfg4_tensor_core_kernel_ragged_members_and_episodes(pop, episodes):
    """Populations that do not fill the four teams of a block, episode counts that leave a partial
    episode block, and more items than resident teams (1186 > 2 * 592: teams loop three times)."""
    w = W.CFG4.with_(pop_size=pop, episodes=episodes)
    members = sorted({0, 1, pop // 2, pop - 1})
    T = 40 if pop > 100 else 120
    _rollout_check(w, T, members, ROLLOUT_AUTO, check_trace=pop <= 100)


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_TILED, ROLLOUT_AUTO])
def test_cfg4_action_scale_and_later_generation(kernel):
    """An action scale other than 1 and the initial states of a later generation (the roll-out seeds
    depend on the generation counter) through all three kernels of the tanh-linear task."""
    w = W.CFG4.with_(pop_size=6, action_scale=0.5, horizon=80)
    s = Solver(w, rollout_kernel=kernel)
    for gen in range(2):
        theta = s.ask().cpu().numpy()
        fit = s.rollout().cpu().numpy()
        fit_o, _ = oracle_fitness(w, theta, gen, 80)
        assert rel_err(fit, fit_o, floor=1.0) < FIT_TOL, gen
        s.tell(torch.tensor(fit, device="cuda"))
    assert s.sync_status() == 0
    s.close()


def test_cfg4_tensor_core_kernel_with_weights_beyond_the_fp16_range():
    """The tensor-core kernel holds the wide layers as fp16 pairs; a weight beyond +-65,504 is clamped
    to that when staged.  The tanh behind it is saturated either way, so the fitness still agrees with
    the oracle (which uses the weight as it is), and nothing turns into an infinity."""
    w = W.CFG4.with_(pop_size=4, horizon=60)
    theta = W.random_parameters(11, 4, w.param_dim, scale=0.05)
    theta[0, 5] = 1.0e7                      # first layer, unit 0
    theta[1, 28 * 128 + 128 + 300] = -3.0e6  # second layer
    theta[2, 7] = 70000.0
    s = Solver(w, rollout_kernel=ROLLOUT_AUTO)
    arg = s.padded_rows(4); arg[:, :w.param_dim] = torch.tensor(theta, device="cuda")
    fit = s.rollout(arg).cpu().numpy()
    assert s.sync_status() == 0 and np.isfinite(fit).all()
    fit_o, _ = oracle_fitness(w, theta, 0, 60)
    assert rel_err(fit, fit_o, floor=1.0) < FIT_TOL
    s.close()


def test_cfg4_tensor_core_and_fp32_kernels_agree_and_repeat():
    w = W.CFG4.with_(pop_size=600, horizon=100)
    a = Solver(w, rollout_kernel=ROLLOUT_AUTO)
    b = Solver(w, rollout_kernel=ROLLOUT_TILED)
    a.ask(); b.ask()
    fa = a.rollout().clone(); fa2 = a.rollout().clone(); fb = b.rollout().clone()
    assert torch.equal(fa, fa2)                                    # run-to-run bitwise
    assert rel_err(fa.cpu().numpy(), fb.cpu().numpy(), floor=1.0) < 1e-4
    assert a.sync_status() == 0 and b.sync_status() == 0
    a.close(); b.close()


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_TILED, ROLLOUT_AUTO])
def test_cfg4_random_policies(kernel):
    w = W.CFG4.with_(pop_size=8)
    theta = W.random_parameters(2, 8, w.param_dim, scale=0.05)   # contracting closed loop
    _rollout_check(w, 100, list(range(8)), kernel, theta_np=theta)


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_AUTO])
def test_zero_policy_is_the_free_pendulum(kernel):
    theta = np.zeros((16, 385), dtype=np.float32)
    _rollout_check(W.CFG1, 150, [0, 15], kernel, theta_np=theta)


def test_generic_kernel_odd_shapes_and_episode_counts():
    # 3 layers of odd widths, episodes not a multiple of the episode block
    sizes = (5, 7, 3, 9, 1)
    w = W.CFG1.with_(layer_sizes=sizes, param_dim=W.mlp_param_count(sizes), pop_size=6, episodes=37,
                     task_param=(1.0, 0.1, 0.5, 9.8, 0.01, 0.2))
    theta = W.random_parameters(3, 6, w.param_dim, scale=0.6)
    _rollout_check(w, 50, list(range(6)), ROLLOUT_GENERIC, theta_np=theta)
    sizes = (28, 8)
    w = W.CFG4.with_(layer_sizes=sizes, param_dim=W.mlp_param_count(sizes), pop_size=4, episodes=3)
    theta = W.random_parameters(4, 4, w.param_dim, scale=0.3)
    _rollout_check(w, 30, list(range(4)), ROLLOUT_GENERIC, theta_np=theta)


@pytest.mark.parametrize("episodes", [5, 8, 9, 37])
def test_cfg2_shape_tiled_variants_and_ragged_episode_counts(episodes):
    # <= 8 episodes: one group per block; more: the two-group warp-specialised kernel, incl. ragged tails
    w = W.CFG2.with_(pop_size=6, episodes=episodes)
    theta = W.random_parameters(7, 6, w.param_dim, scale=0.3)
    _rollout_check(w, 60, list(range(6)), ROLLOUT_TILED, theta_np=theta)


@pytest.mark.parametrize("hidden", [32, 128])
@pytest.mark.parametrize("episodes", [3, 16, 21])
def test_other_cartpole_widths_have_fast_kernels(hidden, episodes):
    sizes = (5, hidden, hidden, 1)
    w = W.CFG2.with_(pop_size=6, episodes=episodes, layer_sizes=sizes, param_dim=W.mlp_param_count(sizes))
    theta = W.random_parameters(hidden, 6, w.param_dim, scale=0.25)
    _rollout_check(w, 60, list(range(6)), ROLLOUT_TILED, theta_np=theta)


@pytest.mark.parametrize("sizes,kernel", [((5, 48, 48, 1), ROLLOUT_TILED), ((5, 20, 50, 1), ROLLOUT_TILED),
                                          ((5, 100, 7, 1), ROLLOUT_AUTO), ((28, 96, 96, 8), ROLLOUT_AUTO),
                                          ((28, 96, 96, 8), ROLLOUT_TILED), ((28, 40, 120, 8), ROLLOUT_AUTO)])
def test_policies_narrower_than_a_compiled_shape_run_on_its_fast_kernel(sizes, kernel):
    """Any two-hidden-layer policy whose hidden widths fit a compiled shape runs on that shape's kernel
    with the missing rows and columns as zeros (TILED is refused when no fast kernel applies, so a
    pass also shows that the fast path was taken)."""
    base = W.CFG2 if sizes[0] == 5 else W.CFG4
    w = base.with_(pop_size=6, episodes=16 if sizes[0] == 5 else 4, layer_sizes=sizes, param_dim=W.mlp_param_count(sizes))
    theta = W.random_parameters(sum(sizes), 6, w.param_dim, scale=0.25 if sizes[0] == 5 else 0.05)
    _rollout_check(w, 60, list(range(6)), kernel, theta_np=theta)


def _rollout_ms(w, kernel, repeats=3):
    s = Solver(w, rollout_kernel=kernel)
    s.ask()
    fit = torch.empty(w.pop_size, device="cuda")
    s.rollout(fitness=fit)
    best = 1e9
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); s.rollout(fitness=fit); e1.record(); e1.synchronize()
        best = min(best, e0.elapsed_time(e1))
    assert s.sync_status() == 0
    s.close()
    return best


@pytest.mark.parametrize("base,narrow,wide", [(W.CFG2, (5, 48, 48, 1), (5, 64, 64, 1)),
                                               (W.CFG4, (28, 96, 96, 8), (28, 128, 128, 8))])
def test_narrower_policies_run_within_twice_the_time_of_the_compiled_shape(base, narrow, wide):
    """A 5-48-48-1 and a 28-96-96-8 policy at the full population must not fall back to the slow
    runtime-shape kernel: their roll-out takes at most twice as long as the compiled shape's."""
    T = 200
    t_narrow = _rollout_ms(base.with_(horizon=T, layer_sizes=narrow, param_dim=W.mlp_param_count(narrow)), ROLLOUT_AUTO)
    t_wide = _rollout_ms(base.with_(horizon=T, layer_sizes=wide, param_dim=W.mlp_param_count(wide)), ROLLOUT_AUTO)
    assert t_narrow < 2.0 * t_wide, (t_narrow, t_wide)


def test_cfg1_shape_with_several_episodes():
    w = W.CFG1.with_(episodes=3)
    _rollout_check(w, 80, list(range(16)), ROLLOUT_TILED)


def test_rollout_later_generation_uses_new_initial_states():
    w = W.CFG1.with_(horizon=50)
    s = Solver(w)
    f = []
    for gen in range(2):
        theta = s.ask()
        fit = s.rollout()
        fit_o, _ = oracle_fitness(w, theta.cpu().numpy(), gen, 50)
        assert rel_err(fit.cpu().numpy(), fit_o, floor=1.0) < FIT_TOL
        s.tell(fit)
        f.append(fit.cpu().numpy())
    assert s.sync_status() == 0
    s.close()


def test_full_horizon_reward_bounds_and_determinism():
    for w in (W.CFG2.with_(pop_size=32), W.CFG4.with_(pop_size=64)):
        s = Solver(w)
        s.ask()
        a = s.rollout().clone()
        b = s.rollout().clone()
        assert torch.equal(a, b)
        a = a.cpu().numpy()
        if w.task_kind == W.TASK_CARTPOLE:
            assert np.abs(a).max() <= w.horizon
        else:
            assert a.max() <= 0 and np.isfinite(a).all()
        s.close()
