"""Parity of the triangle-painting roll-out (paper Section 3, "Concrete and Abstract Painting") with
the oracle through the C-ABI: coverage bit for bit, colours and fitness to fp32 rounding."""
import numpy as np
import pytest
import torch

import oracle
from paper_2202_05008_b200 import Solver, EvoError, workloads as W
from paper_2202_05008_b200.train import run

pytestmark = pytest.mark.gpu


def _workload(n_tri, width, height, P, sigma=0.6, bg=0.0, seed=21):
    return W.PAINT.with_(pop_size=P, param_dim=10 * n_tri, sigma=sigma, seed=seed,
                         task_param=(float(width), float(height), float(bg)))


def _render(w, theta=None, want_canvas=True):
    width, height = int(w.task_param[0]), int(w.task_param[1])
    s = Solver(w, trace_steps=1 if want_canvas else 0)
    target = torch.tensor(W.paint_target(w.seed, width, height), device="cuda")
    s.set_target(target)
    if theta is None:
        th = s.ask()
        arg = None
    else:
        s.ask()
        arg = s.padded_rows(w.pop_size); arg[:, :w.param_dim] = torch.tensor(theta, device="cuda")
        th = arg[:, :w.param_dim]
    canvas = torch.zeros(w.pop_size, height, width, 3, device="cuda") if want_canvas else None
    fit = s.rollout(theta=arg, trace=canvas).cpu().numpy()
    assert s.sync_status() == 0
    return th.cpu().numpy(), fit, (canvas.cpu().numpy() if want_canvas else None), target.cpu().numpy()


@pytest.mark.parametrize("n_tri,width,height,bg", [(20, 70, 45, 0.0), (7, 32, 16, 0.25), (130, 33, 129, 1.0)])
def test_canvas_and_fitness_match_oracle(n_tri, width, height, bg):
    w = _workload(n_tri, width, height, P=6, bg=bg)
    theta, fit, canvas, target = _render(w)
    for m in range(w.pop_size):
        want = oracle.paint_render(theta[m].reshape(-1, 10), width, height, bg)
        assert np.max(np.abs(canvas[m] - want)) < 2e-6 * max(1, n_tri // 8)
        # pixels no triangle touched keep the background bit for bit, on both sides the same ones
        assert np.array_equal(np.all(canvas[m] == np.float32(bg), axis=-1), np.all(want == np.float64(np.float32(bg)), axis=-1))
        f = oracle.paint_fitness(theta[m].reshape(-1, 10), width, height, target, bg)
        assert abs(fit[m] - f) < 1e-6


def test_coverage_is_bit_exact_for_opaque_single_triangles_needles_included():
    rng = np.random.default_rng(8)
    P, width, height = 96, 61, 47
    theta = np.zeros((P, 10), np.float32)
    theta[:, :6] = rng.uniform(-1.3, 1.3, (P, 6))
    # needles: third vertex almost on the segment between the other two
    for m in range(0, P, 3):
        s = rng.random()
        theta[m, 4:6] = theta[m, 0:2] + s * (theta[m, 2:4] - theta[m, 0:2]) + rng.normal(0, 1e-6, 2)
    theta[:, 6:10] = 5.0                                         # white, opaque after clamping
    w = _workload(1, width, height, P=P)
    _, _, canvas, _ = _render(w, theta)
    covered = 0
    for m in range(P):
        want = oracle.paint_render(theta[m][None], width, height) == 1.0
        assert np.array_equal(canvas[m] == 1.0, want)
        covered += int(want[:, :, 0].sum())
    assert covered > 10000


def test_full_size_workload_sampled_members_and_repeatability():
    w = W.PAINT
    s = Solver(w)
    target = torch.tensor(W.paint_target(w.seed, 128, 128), device="cuda")
    s.set_target(target)
    theta = s.ask()
    a = s.rollout().clone(); b = s.rollout().clone()
    assert torch.equal(a, b)
    for m in (0, 1, 511, 1023):
        f = oracle.paint_fitness(theta[m].cpu().numpy().reshape(-1, 10), 128, 128, target.cpu().numpy(), 0.0)
        assert abs(float(a[m]) - f) < 1e-6
    assert s.sync_status() == 0


def test_order_and_argument_errors():
    w = _workload(4, 16, 16, P=2)
    s = Solver(w)
    s.ask()
    with pytest.raises(EvoError):
        s.rollout()                                              # no target bound
    with pytest.raises(EvoError):
        Solver(w.with_(param_dim=41))                            # not a whole number of triangles
    with pytest.raises(EvoError):
        Solver(w.with_(task_param=(16.5, 16.0, 0.0)))
    with pytest.raises(EvoError):
        Solver(W.CFG1).set_target(torch.zeros(4, 4, 3, device="cuda"))


def test_painting_gets_closer_to_the_target():
    w = W.PAINT.with_(pop_size=256, task_param=(64.0, 64.0, 0.0))
    target = torch.tensor(W.paint_target(w.seed, 64, 64), device="cuda")
    _, hist = run(w, 150, target=target)
    assert hist[-1][0] > hist[0][0] + 0.01 and hist[-1][0] > -0.06
