"""The checked build of the library (libevo_debug.so, -DEVO_DEBUG) on the tiny and odd-sized cases.

No memory checker can be run on the kernels, so the library has a build in which every workspace
region is followed by guard bytes and the kernels' global stores test their index first.  Here the
smallest populations, every parameter count from 1 to 9 (ragged 128-bit stores), horizons of 1 to 3
steps and odd episode counts run through that build; after every call the guard bytes must be
intact and no store may have been skipped, and the results must still agree with the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err, oracle_fitness
from paper_2202_05008_b200 import Solver, EvoError, workloads as W
from paper_2202_05008_b200 import build as B
from paper_2202_05008_b200.binding import ROLLOUT_GENERIC, ROLLOUT_AUTO

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    B.build_library(debug=True)


def _clean(s):
    assert s.debug_check() == (-1, 0, 0)


@pytest.mark.parametrize("D", list(range(1, 10)) + [31, 32, 33])
@pytest.mark.parametrize("noise", [W.NOISE_STORED, W.NOISE_REGENERATED])
def test_ask_tell_on_the_smallest_population_and_every_small_parameter_count(D, noise):
    w = W.Workload("tiny", 2, D, seed=D, sigma=0.1)
    s = Solver(w, debug=True, noise_mode=noise)
    for gen in range(2):
        theta = s.ask()
        _clean(s)
        th_o, eps_o = oracle.ask(w.seed, gen, 2, D, s.center().cpu().numpy(), w.sigma)
        assert (theta.cpu().numpy().view(np.uint32) == th_o.view(np.uint32)).all()
        s.tell(torch.tensor([0.5 + gen, -1.0], device="cuda"))
        _clean(s)
    assert s.sync_status() == 0
    s.close()


@pytest.mark.parametrize("T", [1, 2, 3])
@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_AUTO])
def test_rollouts_of_one_to_three_steps_with_traces(T, kernel):
    for w in (W.CFG1.with_(pop_size=2, horizon=T), W.CFG2.with_(pop_size=2, episodes=3, horizon=T),
              W.CFG2.with_(pop_size=4, episodes=11, horizon=T), W.CFG4.with_(pop_size=2, episodes=5, horizon=T)):
        s = Solver(w, debug=True, trace_steps=T, rollout_kernel=kernel)
        theta = s.ask().cpu().numpy()
        sd = 4 if w.task_kind == W.TASK_CARTPOLE else 28
        trace = torch.zeros(w.pop_size, w.episodes, T, sd, device="cuda")
        fit = s.rollout(trace=trace).cpu().numpy()
        _clean(s)
        fit_o, _ = oracle_fitness(w, theta, 0, T)
        assert rel_err(fit, fit_o, floor=1.0) < 1e-3
        s.tell(torch.tensor(fit, device="cuda"))
        _clean(s)
        assert s.sync_status() == 0
        s.close()


def test_single_step_tasks_and_sharded_tell_leave_the_guards_intact():
    w = W.CFG3.with_(pop_size=2, batch=3)
    s = Solver(w, debug=True)
    images, labels = W.image_batch(w.seed, 0, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    s.ask(); fit = s.rollout(); _clean(s)
    s.tell(fit); _clean(s)
    s.close()
    ws = W.SEQ2SEQ.with_(pop_size=2, batch=5)
    s = Solver(ws, debug=True)
    s.ask(); fit = s.rollout(); _clean(s)
    s.close()
    wp = W.PAINT.with_(pop_size=2)
    s = Solver(wp, debug=True)
    s.set_target(torch.tensor(W.paint_target(wp.seed, 128, 128), device="cuda"))
    s.ask(); fit = s.rollout(); _clean(s)
    s.close()
    w1 = W.CFG1.with_(pop_size=6, horizon=2, sigma_mode=W.SIGMA_PGPE, optimizer=W.OPT_CLIPUP)
    s = Solver(w1, debug=True, shard_first_pair=1, shard_pairs=2)
    s.ask(); fit = s.rollout(); _clean(s)
    s.tell_begin(torch.zeros(6, device="cuda").normal_()); _clean(s)
    s.tell_end(); _clean(s)
    assert s.sync_status() == 0
    s.close()


def test_a_changed_guard_byte_is_reported_and_the_normal_build_has_no_check():
    """The host-side check itself: overwrite one guard byte of the last region from the host (it is the
    caller's memory) and see it reported; the normal build answers UNSUPPORTED."""
    w = W.Workload("tiny", 4, 5, seed=1, sigma=0.1)
    s = Solver(w, debug=True)
    s.ask()
    _clean(s)
    off = s._ws_ptr - s.workspace.data_ptr() + s.workspace_bytes - 1      # last byte = last guard byte
    assert int(s.workspace[off]) == 0xA5
    s.workspace[off] = 0
    region, site, _ = s.debug_check()
    assert region >= 0 and site == 0
    s.workspace[off] = 0xA5
    _clean(s)
    s.close()
    plain = Solver(w)
    with pytest.raises(EvoError) as e:
        plain.debug_check()
    assert e.value.code == 7
    plain.close()
