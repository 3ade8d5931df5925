"""Parity at the full sizes and launch configurations that bench.py times, on sampled outputs."""
import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err, oracle_fitness
from paper_2202_05008_b200 import Solver, workloads as W

pytestmark = pytest.mark.gpu


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 2**30


@pytest.mark.parametrize("noise_mode", [W.NOISE_STORED, W.NOISE_REGENERATED])
def test_update_sweep_full_size_sampled_columns(noise_mode):
    w = W.CFG5
    need = 100 if noise_mode == W.NOISE_STORED else 68
    torch.cuda.empty_cache()
    if _free_gb() < need + 8:
        pytest.skip(f"needs {need} GiB of free device memory")
    P, D, H = w.pop_size, w.param_dim, w.pop_size // 2
    s = Solver(w, noise_mode=noise_mode)
    theta = s.ask()
    quads = [0, 131071, 262143]                       # first, middle and last column quad
    cols = np.concatenate([np.arange(4 * q, 4 * q + 4) for q in quads])
    th = theta[:, torch.tensor(cols, device="cuda")].cpu().numpy()          # [P][12]
    eps_o = np.zeros((H, len(cols)), dtype=np.float32)
    for j in range(H):
        for i, q in enumerate(quads):
            eps_o[j, 4 * i:4 * i + 4] = oracle.normal4(oracle.stream_words(w.seed, 0, 0, j, q))
    sig = np.float32(w.sigma)
    assert (th[0::2].view(np.uint32) == (sig * eps_o).view(np.uint32)).all()
    assert (th[1::2].view(np.uint32) == (-sig * eps_o).view(np.uint32)).all()
    if noise_mode == W.NOISE_STORED:
        eps = s.eps()[:, torch.tensor(cols, device="cuda")].cpu().numpy()
        assert (eps.view(np.uint32) == eps_o.view(np.uint32)).all()
    f = W.synthetic_fitness(w.seed, 0, P)
    s.tell(torch.tensor(f, device="cuda"))
    assert s.sync_status() == 0
    rank, u = (x.cpu().numpy() for x in s.ranks())
    rank_o, u_o, bad = oracle.centered_rank(f)
    assert not bad and (rank == rank_o).all() and (u.view(np.uint32) == u_o.view(np.uint32)).all()
    g_o = oracle.gradient(u_o, eps_o, float(sig))
    g = s.gradient()[torch.tensor(cols, device="cuda")].cpu().numpy()
    assert rel_err(g, g_o) < 1e-5
    z = np.zeros(len(cols))
    c_o, m_o, v_o = oracle.adam(z, z, z, g_o, 1, float(np.float32(w.lr)), float(np.float32(0.9)),
                                float(np.float32(0.999)), float(np.float32(1e-8)))
    c = s.center()[torch.tensor(cols, device="cuda")].cpu().numpy()
    assert rel_err(c, c_o) < 1e-5
    # the whole centre moved by about +-lr (first Adam step), nothing is NaN
    call = s.center()
    assert torch.isfinite(call).all() and float(call.abs().max()) <= 0.0100001
    s.close()
    del s, theta
    torch.cuda.empty_cache()


def test_cfg2_full_population_full_horizon_bounds_and_sampled_parity():
    # the bench configuration (P=256, E=16, T=1000): bounds and determinism at T=1000,
    # parity against the oracle for sampled members at T=200 in the same launch shape
    w = W.CFG2
    s = Solver(w)
    theta = s.ask()
    a = s.rollout().clone(); b = s.rollout().clone()
    assert torch.equal(a, b) and float(a.abs().max()) <= w.horizon
    s.close()
    w200 = w.with_(horizon=200)
    s = Solver(w200)
    th = s.ask().cpu().numpy()
    fit = s.rollout().cpu().numpy()
    members = [0, 37, 100, 255]
    fit_o, _ = oracle_fitness(w200, th[members], 0, 200)
    assert rel_err(fit[members], fit_o, floor=1.0) < 1e-3
    s.close()


def test_cfg4_full_population_full_horizon_bounds_and_sampled_parity():
    # the bench configuration (P=4096, E=4, T=1000) in its launch shape: bounds, determinism, and the
    # fitness of sampled members (first, last, the team/block boundaries of the persistent kernel)
    # against the oracle at the full horizon
    w = W.CFG4
    s = Solver(w)
    theta = s.ask()
    a = s.rollout().clone(); b = s.rollout().clone()
    assert torch.equal(a, b)
    a = a.cpu().numpy()
    assert np.isfinite(a).all() and a.max() <= 0.0 and a.min() >= -(28.08 * w.horizon + 400)
    members = [0, 147, 148, 591, 592, 2047, 4095]
    fit_o, _ = oracle_fitness(w, theta[members].cpu().numpy(), 0, w.horizon)
    assert rel_err(a[members], fit_o, floor=1.0) < 1e-3
    assert s.sync_status() == 0
    s.close()


def test_cfg2_full_horizon_sampled_parity():
    w = W.CFG2
    s = Solver(w)
    theta = s.ask()
    fit = s.rollout().cpu().numpy()
    members = [0, 37, 100, 255]
    fit_o, _ = oracle_fitness(w, theta[members].cpu().numpy(), 0, w.horizon)
    assert rel_err(fit[members], fit_o, floor=1.0) < 1e-3
    s.close()


def test_cfg3_full_batch_every_member():
    w = W.CFG3
    s = Solver(w)
    images, labels = W.image_batch(w.seed, 0, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    th = s.ask().cpu().numpy()
    fit = s.rollout().cpu().numpy()
    assert s.sync_status() == 0
    sub = images[:128], labels[:128]
    # all 64 members against the oracle would take minutes on the full batch; every 8th member is
    # checked on the full batch
    members = list(range(0, 64, 8))
    want = np.array([oracle.cnn_fitness(th[m], images, labels, True) for m in members])
    assert rel_err(fit[members], want, floor=1.0) < 1e-3
    assert np.isfinite(fit).all() and (fit < 0).all()
    s.close()
