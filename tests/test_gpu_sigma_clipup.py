"""Per-dimension sigma with the PGPE sigma update, and the ClipUp optimiser, against the oracle
(teacher-forced per generation: the oracle starts from the GPU's state)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err
from paper_2202_05008_b200 import Solver, workloads as W

pytestmark = pytest.mark.gpu
F32 = lambda x: float(np.float32(x))


def _fitness(w, gen):
    return W.synthetic_fitness(w.seed, gen, w.pop_size)


@pytest.mark.parametrize("noise_mode", [W.NOISE_STORED, W.NOISE_REGENERATED])
@pytest.mark.parametrize("P,D", [(16, 385), (258, 130), (4096, 1000)])
def test_pgpe_sigma_update_three_generations(noise_mode, P, D):
    w = W.Workload("sigma", P, D, seed=P + D, sigma=0.1, sigma_mode=W.SIGMA_PGPE)
    s = Solver(w, noise_mode=noise_mode)
    assert torch.equal(s.sigma(), torch.full((D,), np.float32(0.1), device="cuda"))
    for gen in range(3):
        sg0 = s.sigma().cpu().numpy()
        c0 = s.center().cpu().numpy()
        m0, v0 = (x.cpu().numpy().astype(np.float64) for x in s.moments())
        theta = s.ask().cpu().numpy()
        th_o, eps_o = oracle.ask_sigma(w.seed, gen, P, D, c0, sg0)
        assert (theta.view(np.uint32) == th_o.view(np.uint32)).all()
        f = _fitness(w, gen)
        s.tell(torch.tensor(f, device="cuda"))
        assert s.sync_status() == 0
        _, u_o, _ = oracle.centered_rank(f)
        g_o = oracle.gradient_sigma(u_o, eps_o, sg0.astype(np.float64))
        assert rel_err(s.gradient().cpu().numpy(), g_o) < 1e-5
        c_o, _, _ = oracle.adam(c0.astype(np.float64), m0, v0, g_o, gen + 1, F32(w.lr), F32(0.9), F32(0.999), F32(1e-8))
        keep = np.abs(g_o) >= 1e-6 * np.sqrt(np.mean(g_o ** 2))
        assert rel_err(s.center().cpu().numpy()[keep], c_o[keep]) < 1e-5
        gs_o = oracle.sigma_gradient(u_o, eps_o, sg0.astype(np.float64))
        sg_o = oracle.sigma_update(sg0.astype(np.float64), gs_o, F32(0.1), F32(0.2))
        sg = s.sigma().cpu().numpy()
        assert rel_err(sg, sg_o) < 1e-5
        assert (sg > 0).all() and (np.abs(sg / sg0 - 1.0) <= 0.2 + 1e-6).all()
        assert not np.array_equal(sg, sg0)
    # padding columns of sigma stay zero
    full = s._view_f32(s.sigma().data_ptr(), 1, s.ldD)[0]
    assert (full[D:] == 0).all()
    s.close()


def test_sigma_clip_limits_the_relative_change():
    w = W.Workload("sigma", 64, 40, seed=5, sigma=0.1, sigma_mode=W.SIGMA_PGPE, sigma_lr=50.0, sigma_max_change=0.1)
    s = Solver(w)
    s.ask(); s.tell(torch.tensor(_fitness(w, 0), device="cuda"))
    ratio = s.sigma().cpu().numpy() / np.float32(0.1)
    at_limit = (np.abs(ratio - 0.9) < 1e-5) | (np.abs(ratio - 1.1) < 1e-5)
    assert at_limit.mean() > 0.8 and (ratio > 0.9 - 1e-5).all() and (ratio < 1.1 + 1e-5).all()
    s.close()


def test_constant_sigma_mode_never_touches_sigma_and_set_sigma_round_trips():
    w = W.Workload("sigma", 32, 50, seed=6, sigma=0.3)
    s = Solver(w)
    s.ask(); s.tell(torch.tensor(_fitness(w, 0), device="cuda"))
    assert torch.equal(s.sigma(), torch.full((50,), np.float32(0.3), device="cuda"))
    new = torch.linspace(0.05, 0.5, 50, device="cuda")
    s.set_sigma(new)
    c0 = s.center().cpu().numpy()
    theta = s.ask().cpu().numpy()
    th_o, _ = oracle.ask_sigma(w.seed, 1, 32, 50, c0, new.cpu().numpy())
    assert (theta.view(np.uint32) == th_o.view(np.uint32)).all()
    s.close()


@pytest.mark.parametrize("noise_mode", [W.NOISE_STORED, W.NOISE_REGENERATED])
@pytest.mark.parametrize("P,D,lr,vmax", [(16, 385, 0.01, 0.0), (64, 5000, 0.05, 0.06), (512, 33, 0.2, 0.25)])
def test_clipup_three_generations(noise_mode, P, D, lr, vmax):
    w = W.Workload("clipup", P, D, seed=P * 3 + D, sigma=0.1, lr=lr, optimizer=W.OPT_CLIPUP, clipup_max_speed=vmax)
    max_speed = F32(vmax) if vmax else 2.0 * F32(lr)
    s = Solver(w, noise_mode=noise_mode)
    clipped = 0
    for gen in range(3):
        c0 = s.center().cpu().numpy().astype(np.float64)
        v0 = s.moments()[0].cpu().numpy().astype(np.float64)           # velocity lives in the m buffer
        s.ask()
        f = _fitness(w, gen)
        s.tell(torch.tensor(f, device="cuda"))
        assert s.sync_status() == 0
        _, eps_o = oracle.ask(w.seed, gen, P, D, np.zeros(D, np.float32), w.sigma)
        _, u_o, _ = oracle.centered_rank(f)
        g_o = oracle.gradient(u_o, eps_o, F32(w.sigma))
        assert rel_err(s.gradient().cpu().numpy(), g_o) < 1e-5
        c_o, v_o = oracle.clipup(c0, v0, g_o, F32(lr), F32(0.9), max_speed)
        assert rel_err(s.moments()[0].cpu().numpy(), v_o) < 1e-5
        assert rel_err(s.center().cpu().numpy(), c_o) < 1e-5
        vn = float(np.linalg.norm(s.moments()[0].cpu().numpy().astype(np.float64)))
        assert vn <= max_speed * (1 + 1e-5)
        clipped += vn > max_speed * (1 - 1e-4)
        if gen == 0:
            assert abs(vn - min(F32(lr), max_speed)) < 1e-5 * F32(lr)   # first step has length lr
    if vmax and vmax < 1.9 * lr:
        assert clipped >= 1                                             # the speed limit was active
    assert s.counters() == (3, 3)
    s.close()


def test_clipup_nan_fitness_skips_the_step():
    w = W.Workload("clipup", 16, 20, seed=1, sigma=0.1, optimizer=W.OPT_CLIPUP)
    s = Solver(w)
    s.ask(); s.tell(torch.tensor(_fitness(w, 0), device="cuda"))
    c1 = s.center().clone(); v1 = s.moments()[0].clone()
    s.ask(); f = _fitness(w, 1); f[3] = np.nan
    s.tell(torch.tensor(f, device="cuda"))
    assert s.sync_status() == 5
    assert torch.equal(s.center(), c1) and torch.equal(s.moments()[0], v1)
    s.close()
