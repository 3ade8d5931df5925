"""ask on the GPU against the oracle: bit-exact noise and parameters."""
import numpy as np
import pytest
import torch

import oracle
from paper_2202_05008_b200 import Solver, workloads as W

pytestmark = pytest.mark.gpu


def _check_ask(w, generations=1, rows=None, stored=True):
    s = Solver(w, noise_mode=W.NOISE_STORED if stored else W.NOISE_REGENERATED)
    center = np.zeros(w.param_dim, dtype=np.float32)
    for gen in range(generations):
        theta = s.ask()
        th = theta.cpu().numpy()
        eps = s.eps().cpu().numpy() if stored else None
        if gen > 0:
            center = s.center().cpu().numpy()
        pairs = range(w.pop_size // 2) if rows is None else rows
        for j in pairs:
            e = oracle.eps_row(w.seed, gen, j, w.param_dim)
            sig = np.float32(w.sigma)
            plus = (sig.astype(np.float64) * e.astype(np.float64) + center).astype(np.float32)
            minus = (-sig.astype(np.float64) * e.astype(np.float64) + center).astype(np.float32)
            if stored:
                assert (eps[j].view(np.uint32) == e.view(np.uint32)).all(), (gen, j)
            assert (th[2 * j].view(np.uint32) == plus.view(np.uint32)).all(), (gen, j)
            assert (th[2 * j + 1].view(np.uint32) == minus.view(np.uint32)).all(), (gen, j)
        # padding columns are zero
        full = s._view_f32(theta.data_ptr(), w.pop_size, s.ldD)
        assert (full[:, w.param_dim:] == 0).all()
        if generations > 1:
            f = torch.tensor(W.synthetic_fitness(w.seed, gen, w.pop_size), device="cuda")
            s.tell(f)
    assert s.sync_status() == 0
    s.close()


def test_ask_cfg1_bitwise_against_oracle_call():
    w = W.CFG1.with_(task_kind=W.TASK_NONE, policy_kind=W.POLICY_NONE, layer_sizes=())
    s = Solver(w)
    theta = s.ask().cpu().numpy()
    eps = s.eps().cpu().numpy()
    th_o, eps_o = oracle.ask(w.seed, 0, w.pop_size, w.param_dim, np.zeros(w.param_dim, np.float32), w.sigma)
    assert (theta.view(np.uint32) == th_o.view(np.uint32)).all()
    assert (eps.view(np.uint32) == eps_o.view(np.uint32)).all()
    assert (theta[0::2] + theta[1::2] == 0).all()
    s.close()


@pytest.mark.parametrize("P,D", [(2, 1), (2, 2), (2, 3), (4, 5), (6, 7), (2, 9), (10, 33), (18, 127), (4, 1025)])
def test_ask_ragged_shapes(P, D):
    _check_ask(W.Workload("ragged", P, D, seed=7 + D, sigma=0.3), generations=3)


def test_ask_cfg2_three_generations_nonzero_centre():
    _check_ask(W.CFG2.with_(task_kind=W.TASK_NONE, policy_kind=W.POLICY_NONE, layer_sizes=()), generations=3)


def test_ask_regenerated_mode_has_no_eps_and_same_theta():
    _check_ask(W.CFG1.with_(task_kind=W.TASK_NONE, policy_kind=W.POLICY_NONE, layer_sizes=()),
               generations=2, stored=False)


def test_ask_cfg4_sampled_pairs():
    w = W.CFG4.with_(task_kind=W.TASK_NONE, policy_kind=W.POLICY_NONE, layer_sizes=())
    _check_ask(w, generations=1, rows=[0, 1, 777, 2047])
