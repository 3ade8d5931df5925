"""Pair-sharded generation (paper Section 2, device parallelism): W solvers, each owning a
contiguous range of antithetic pairs, must reproduce the unsharded solver.  The shards run one
after the other on one device and their reduce buffers are summed by hand, which is what the
all-reduce does between ranks; no kernel waits on another."""
import numpy as np
import pytest
import torch

from paper_2202_05008_b200 import binding, workloads as W
from helpers import rel_err

pytestmark = pytest.mark.gpu


def _shards(w, world, **kw):
    H = w.pop_size // 2
    per = H // world
    return [binding.Solver(w, shard_first_pair=r * per, shard_pairs=per, **kw) for r in range(world)]


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("noise", [W.NOISE_STORED, W.NOISE_REGENERATED])
def test_sharded_cartpole_generations_match_unsharded(world, noise):
    w = W.CFG1.with_(pop_size=64)
    full = binding.Solver(w, noise_mode=noise)
    shards = _shards(w, world, noise_mode=noise)
    for gen in range(3):
        theta_full = full.ask().clone()
        fit_full = full.rollout().clone()
        full.tell(fit_full)
        # shard r's rows are rows [2 first_pair, 2 (first_pair + pairs)) of the full population
        theta_sh = torch.cat([s.ask() for s in shards])
        assert torch.equal(theta_sh, theta_full)
        fits = [s.rollout().clone() for s in shards]
        fit_all = torch.cat(fits)
        assert torch.equal(fit_all, fit_full)
        for s in shards:
            s.tell_begin(fit_all)
        bufs = [s.reduce_buffers() for s in shards]
        g = torch.stack([b[0] for b in bufs]).sum(0)
        for s, b in zip(shards, bufs):
            b[0].copy_(g)
            s.tell_end()
        c_full = full.center().cpu().numpy()
        for s in shards:
            assert rel_err(s.center().cpu().numpy(), c_full) < 1e-6
            assert rel_err(s.gradient().cpu().numpy(), full.gradient().cpu().numpy()) < 1e-6
        # every shard holds bit-identical state
        for s in shards[1:]:
            assert torch.equal(s.center(), shards[0].center())
    assert all(s.sync_status() == 0 for s in shards) and full.sync_status() == 0


def _sharded_generation_by_hand(shards, fit_all=None):
    """ask -> rollout -> tell on every shard in turn, the two exchanges done by hand: fitness shards
    concatenated in member order, reduce buffers summed and handed back to every shard."""
    thetas = [s.ask() for s in shards]
    if fit_all is None:
        fit_all = torch.cat([s.rollout().clone() for s in shards])
    for s in shards:
        s.tell_begin(fit_all)
    bufs = [s.reduce_buffers() for s in shards]
    g = torch.stack([b[0] for b in bufs]).sum(0)
    for s, b in zip(shards, bufs):
        b[0].copy_(g)
        s.tell_end()
    return thetas, fit_all


@pytest.mark.parametrize("world", [2, 8])
def test_sharded_large_population_tanh_linear_matches_unsharded(world):
    """The large-population control configuration (4,096 members, MLP 28-128-128-8, 4 episodes) in
    pair shards, horizon cut to 50 steps: rows and fitness bit-equal to the unsharded solver, centre
    within 1e-6, shards bit-identical among themselves."""
    w = W.CFG4.with_(horizon=50)
    full = binding.Solver(w)
    theta_full = full.ask()
    fit_full = full.rollout().clone()
    full.tell(fit_full)
    shards = _shards(w, world)
    thetas, fit_all = _sharded_generation_by_hand(shards)
    per = w.pop_size // world
    for r in (0, world - 1):                                        # first and last shard's rows
        assert torch.equal(thetas[r], theta_full[r * per:(r + 1) * per])
    assert torch.equal(fit_all, fit_full)
    c_full = full.center().cpu().numpy()
    for s in shards:
        assert rel_err(s.center().cpu().numpy(), c_full) < 1e-6
    for s in shards[1:]:
        assert torch.equal(s.center(), shards[0].center())
    assert all(s.sync_status() == 0 for s in shards) and full.sync_status() == 0
    for s in shards:
        s.close()
    full.close()


@pytest.mark.parametrize("world", [2, 8])
def test_sharded_update_sweep_with_regenerated_noise_matches_unsharded(world):
    """The update-bandwidth configuration (16,384 members, no task, regenerated noise) at a reduced
    parameter count (D = 8,200, not a multiple of 32): every shard recomputes the noise of its own
    pairs from the global pair index in ask and again in tell."""
    w = W.CFG5.with_(param_dim=8200)
    full = binding.Solver(w, noise_mode=W.NOISE_REGENERATED)
    shards = _shards(w, world, noise_mode=W.NOISE_REGENERATED)
    per = w.pop_size // world
    for gen in range(2):
        fit = torch.tensor(W.synthetic_fitness(w.seed, gen, w.pop_size), device="cuda")
        theta_full = full.ask()
        full.tell(fit)
        thetas, _ = _sharded_generation_by_hand(shards, fit_all=fit)
        for r in (0, world // 2, world - 1):
            assert torch.equal(thetas[r], theta_full[r * per:(r + 1) * per])
        assert rel_err(shards[0].center().cpu().numpy(), full.center().cpu().numpy()) < 1e-6
        for s in shards[1:]:
            assert torch.equal(s.center(), shards[0].center())
    assert all(s.sync_status() == 0 for s in shards) and full.sync_status() == 0
    for s in shards:
        s.close()
    full.close()


def test_sharded_sigma_adaptation_and_clipup_match_oracle():
    w = W.CFG1.with_(pop_size=32, optimizer=W.OPT_CLIPUP, sigma_mode=W.SIGMA_PGPE,
                            sigma_lr=0.2, sigma_max_change=0.2, lr=0.15, clipup_max_speed=0.3)
    full = binding.Solver(w)
    shards = _shards(w, 2)
    rng = np.random.default_rng(5)
    for gen in range(3):
        fit = torch.from_numpy(rng.standard_normal(w.pop_size).astype(np.float32)).cuda()
        full.ask(); full.tell(fit)
        for s in shards:
            s.ask()
        _ = [s.tell_begin(fit) for s in shards]
        bufs = [s.reduce_buffers() for s in shards]
        g = bufs[0][0] + bufs[1][0]
        sg = bufs[0][1] + bufs[1][1]
        for s, b in zip(shards, bufs):
            b[0].copy_(g); b[1].copy_(sg); s.tell_end()
        for s in shards:
            assert rel_err(s.center().cpu().numpy(), full.center().cpu().numpy()) < 1e-5
            assert rel_err(s.sigma().cpu().numpy(), full.sigma().cpu().numpy()) < 1e-5


def test_sharded_supervised_rollout_matches_unsharded():
    w = W.CFG3.with_(pop_size=16, batch=64)
    imgs, labels = W.image_batch(w.seed, 0, w.batch)
    imgs, labels = torch.tensor(imgs, device="cuda"), torch.tensor(labels, device="cuda")
    full = binding.Solver(w)
    full.set_batch(imgs, labels)
    shards = _shards(w, 2)
    for s in shards:
        s.set_batch(imgs, labels)
    full.ask()
    fit_full = full.rollout().clone()
    for s in shards:
        s.ask()
    fit_sh = torch.cat([s.rollout().clone() for s in shards])
    assert torch.equal(fit_sh, fit_full)


def test_sharded_solver_order_and_argument_errors():
    w = W.CFG1.with_(pop_size=16)
    with pytest.raises(RuntimeError):
        binding.Solver(w, shard_first_pair=6, shard_pairs=4)       # runs past the last pair
    s = binding.Solver(w, shard_first_pair=4, shard_pairs=4)
    assert s.P == 8 and s.P_global == 16
    fit = torch.zeros(16, device="cuda")
    with pytest.raises(RuntimeError):
        s.tell_end()                                               # nothing begun
    s.ask()
    with pytest.raises(RuntimeError):
        s.tell(fit)                                                # a shard needs begin/end
    s.tell_begin(fit)
    with pytest.raises(RuntimeError):
        s.tell_begin(fit)
    s.tell_end()
    assert s.counters()[0] == 1
