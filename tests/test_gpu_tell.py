"""tell on the GPU against the oracle: bit-exact ranks, gradient and Adam step."""
import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err
from paper_2202_05008_b200 import Solver, workloads as W

pytestmark = pytest.mark.gpu


def _bare(w):
    return w.with_(task_kind=W.TASK_NONE, policy_kind=W.POLICY_NONE, layer_sizes=())


def _tell_check(w, generations, stored=True, fitness_fn=None):
    """Teacher-forced: every generation the oracle starts from the GPU's state."""
    s = Solver(w, noise_mode=W.NOISE_STORED if stored else W.NOISE_REGENERATED)
    P, D = w.pop_size, w.param_dim
    for gen in range(generations):
        s.ask()
        c0 = s.center().cpu().numpy().astype(np.float64)
        m0, v0 = (x.cpu().numpy().astype(np.float64) for x in s.moments())
        f = (fitness_fn or W.synthetic_fitness)(w.seed, gen, P)
        s.tell(torch.tensor(f, device="cuda"))
        assert s.sync_status() == 0
        rank, u = (x.cpu().numpy() for x in s.ranks())
        rank_o, u_o, bad = oracle.centered_rank(f)
        assert not bad
        assert (rank == rank_o).all()
        assert (u.view(np.uint32) == u_o.view(np.uint32)).all()
        _, eps_o = oracle.ask(w.seed, gen, P, D, np.zeros(D, np.float32), w.sigma)
        g_o = oracle.gradient(u_o, eps_o, float(np.float32(w.sigma)))
        g = s.gradient().cpu().numpy()
        assert rel_err(g, g_o) < 1e-5
        c_o, m_o, v_o = oracle.adam(c0, m0, v0, g_o, gen + 1, float(np.float32(w.lr)),
                                    float(np.float32(0.9)), float(np.float32(0.999)), float(np.float32(1e-8)))
        c = s.center().cpu().numpy()
        keep = np.abs(g_o) >= 1e-6 * np.sqrt(np.mean(g_o ** 2))     # ill-conditioned sign(g) excluded
        assert keep.sum() >= 0.99 * D
        assert rel_err(c[keep], c_o[keep]) < 1e-5
        mm, vv = (x.cpu().numpy() for x in s.moments())
        assert rel_err(mm, m_o) < 1e-5 and rel_err(vv, v_o) < 1e-5
        assert s.counters() == (gen + 1, gen + 1)
    s.close()


def test_tell_cfg1_first_step_is_plus_minus_lr():
    w = _bare(W.CFG1)
    s = Solver(w)
    s.ask()
    s.tell(torch.tensor(W.synthetic_fitness(0, 0, 16), device="cuda"))
    c = s.center().cpu().numpy()
    g = s.gradient().cpu().numpy()
    big = np.abs(g) > 1e-4                    # |step| = lr/(1 + eps/|g|)
    assert big.sum() > 300
    assert np.abs(np.abs(c[big]) - 0.01).max() < 2e-6
    assert (np.sign(c) == np.sign(g)).all()   # ascent
    s.close()


@pytest.mark.parametrize("stored", [True, False])
def test_tell_cfg1_three_generations(stored):
    _tell_check(_bare(W.CFG1), 3, stored)


@pytest.mark.parametrize("P,D", [(2, 1), (4, 3), (6, 7), (34, 33), (258, 130), (1000, 37)])
def test_tell_ragged_shapes(P, D):
    _tell_check(W.Workload("ragged", P, D, seed=P + D, sigma=0.5), 2, True)
    _tell_check(W.Workload("ragged", P, D, seed=P + D, sigma=0.5), 2, False)


def test_tell_cfg2_shape_both_noise_modes():
    _tell_check(_bare(W.CFG2), 2, True)
    _tell_check(_bare(W.CFG2), 2, False)


def test_tell_cfg4_shape_split_reduction():
    _tell_check(_bare(W.CFG4), 1, True)


def test_rank_ties_and_specials_bitwise():
    def fit(seed, gen, P):
        f = np.round(np.random.default_rng(gen).standard_normal(P) * 2).astype(np.float32)  # many ties
        f[3] = np.inf; f[5] = -np.inf; f[7] = 0.0; f[9] = -0.0
        return f
    _tell_check(W.Workload("ties", 4096 + 2, 8, seed=1, sigma=0.5), 2, True, fit)


def test_rank_large_population_split_path():
    # P > 4096 takes the split counting path (integer atomics); ties and specials included
    def fit(seed, gen, P):
        f = np.round(np.random.default_rng(gen + 5).standard_normal(P) * 50).astype(np.float32)
        f[1] = np.inf; f[2] = -np.inf; f[3] = 0.0; f[4] = -0.0
        return f
    _tell_check(W.Workload("bigP", 16384, 40, seed=2, sigma=0.5), 2, True, fit)
    _tell_check(W.Workload("bigP", 5000, 9, seed=3, sigma=0.5), 1, False)
    # NaN is still caught on this path
    w = W.Workload("bigP", 6000, 8, seed=4, sigma=0.5)
    s = Solver(w); s.ask()
    f = W.synthetic_fitness(4, 0, 6000); f[5999] = np.nan
    s.tell(torch.tensor(f, device="cuda"))
    assert s.sync_status() == 5
    s.close()


def test_nan_fitness_skips_the_update_and_is_reported():
    w = _bare(W.CFG1)
    s = Solver(w)
    s.ask()
    s.tell(torch.tensor(W.synthetic_fitness(0, 0, 16), device="cuda"))
    c1 = s.center().clone(); m1, v1 = (x.clone() for x in s.moments())
    s.ask()
    f = W.synthetic_fitness(0, 1, 16); f[11] = np.nan
    s.tell(torch.tensor(f, device="cuda"))
    assert s.sync_status() == 5
    assert s.sync_status() == 0                       # reported once, then cleared
    assert torch.equal(s.center(), c1) and torch.equal(s.moments()[0], m1) and torch.equal(s.moments()[1], v1)
    assert s.counters() == (2, 1)                      # generation advanced, Adam step did not
    s.ask()
    s.tell(torch.tensor(W.synthetic_fitness(0, 2, 16), device="cuda"))
    assert s.sync_status() == 0 and s.counters() == (3, 2)
    assert not torch.equal(s.center(), c1)
    s.close()


def test_call_order_is_enforced():
    from paper_2202_05008_b200 import EvoError
    s = Solver(_bare(W.CFG1))
    f = torch.zeros(16, device="cuda")
    with pytest.raises(EvoError) as e:
        s.tell(f)
    assert e.value.code == 2
    s.ask(); s.tell(f)
    with pytest.raises(EvoError):
        s.tell(f)
    with pytest.raises(EvoError) as e:
        s.rollout()
    assert e.value.code == 7                           # no task configured
    s.close()


def test_checkpoint_resume_is_bitwise():
    w = _bare(W.CFG2.with_(pop_size=64))
    def run(s, g0, n):
        for g in range(g0, g0 + n):
            s.ask(); s.tell(torch.tensor(W.synthetic_fitness(3, g, 64), device="cuda"))
    a = Solver(w); run(a, 0, 4)
    b = Solver(w); run(b, 0, 2)
    gen, t = b.counters()
    c, (m, v) = b.center().clone(), [x.clone() for x in b.moments()]
    b.close()
    r = Solver(w)
    r.set_state(c.contiguous(), m.contiguous(), v.contiguous(), gen, t)
    run(r, 2, 2)
    assert torch.equal(a.center(), r.center())
    assert torch.equal(a.moments()[0], r.moments()[0]) and torch.equal(a.moments()[1], r.moments()[1])
    assert a.counters() == r.counters() == (4, 4)
    # run-to-run determinism of the split reduction
    a2 = Solver(w); run(a2, 0, 4)
    assert torch.equal(a.center(), a2.center())
    a.close(); r.close(); a2.close()
