"""Supervised (CNN) rollout on the GPU against the oracle: fitness within 1e-3."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err
from paper_2202_05008_b200 import Solver, workloads as W
from paper_2202_05008_b200.binding import ROLLOUT_GENERIC, ROLLOUT_AUTO

KERNELS = [ROLLOUT_GENERIC, ROLLOUT_AUTO]      # CUDA-core kernel, tensor-core (tcgen05) path

pytestmark = pytest.mark.gpu


def _run(w, theta_np=None, generation=0, members=None, kernel=ROLLOUT_AUTO):
    s = Solver(w, rollout_kernel=kernel)
    images, labels = W.image_batch(w.seed, generation, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    if theta_np is None:
        theta_np = s.ask().cpu().numpy(); arg = None
    else:
        arg = s.padded_rows(w.pop_size); arg[:, :w.param_dim] = torch.tensor(theta_np, device="cuda")
    fit = s.rollout(arg).cpu().numpy()
    assert s.sync_status() == 0
    members = range(w.pop_size) if members is None else members
    want = np.array([oracle.cnn_fitness(theta_np[m], images, labels, True) for m in members])
    assert rel_err(fit[list(members)], want, floor=1.0) < 1e-3
    s.close()
    return fit


@pytest.mark.parametrize("kernel", KERNELS)
def test_cnn_zero_parameters_is_minus_ln10(kernel):
    w = W.CFG3.with_(pop_size=2, batch=64)
    fit = _run(w, theta_np=np.zeros((2, W.CNN_PARAMS), dtype=np.float32), kernel=kernel)
    assert np.abs(fit + math.log(10)).max() < 1e-6


@pytest.mark.parametrize("kernel", KERNELS)
def test_cnn_cfg3_first_generation_sampled_members(kernel):
    _run(W.CFG3, members=[0, 1, 31, 32, 63], kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_cnn_random_large_parameters_ragged_batch(kernel):
    w = W.CFG3.with_(pop_size=4, batch=77)
    _run(w, theta_np=W.random_parameters(5, 4, W.CNN_PARAMS, scale=0.2), kernel=kernel)


def test_cnn_tensor_core_path_against_the_unrounded_oracle():
    """Against the fp64 oracle with NO bf16 rounding (the mode pinned to torch's conv2d): the bound
    is the kernel's own 1e-3 plus the gap between the two oracle modes, which a CPU test pins
    (tests/test_oracle_bf16_gap.py), so the rounding points the kernel shares with the bf16 oracle
    are bounded by something the kernel did not shape."""
    w = W.CFG3.with_(pop_size=16, batch=256)
    s = Solver(w)
    images, labels = W.image_batch(w.seed, 0, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    theta = s.ask().cpu().numpy()
    fit = s.rollout().cpu().numpy()
    assert s.sync_status() == 0
    members = [0, 1, 7, 8, 15]
    want = np.array([oracle.cnn_fitness(theta[m], images, labels, False) for m in members])
    assert rel_err(fit[members], want, floor=1.0) < 2e-3
    s.close()


def test_cnn_more_than_one_member_group_and_tiny_batch():
    # 70 members = three conv1 groups (32 + 32 + 6); batch 3 = a fifth of one image group
    w = W.CFG3.with_(pop_size=70, batch=3)
    _run(w, theta_np=W.random_parameters(6, 70, W.CNN_PARAMS, scale=0.1), members=[0, 5, 31, 32, 63, 64, 69])


@pytest.mark.parametrize("pop,batch,members", [
    (300, 24, [0, 1, 2, 3, 147, 148, 149, 298, 299]),   # 600 units on 148 blocks: every block runs through 2-3 members
    (296, 16, [0, 1, 2, 3, 100, 295]),                  # one image group per member: every unit is a new member
    (34, 16, [0, 31, 32, 33]),                          # a conv1 group of two members
    (6, 1, [0, 5]),                                     # a single image
    (4, 200, [0, 1, 2, 3]),                             # 13 image groups per member, the last half full
])
def test_cnn_block_ranges_across_members(pop, batch, members):
    """conv2 blocks take contiguous ranges of (member, image group) units: cases where a range runs through
    several members (filter bands restaged in flight), where each unit is a new member, and ragged ends."""
    w = W.CFG3.with_(pop_size=pop, batch=batch)
    _run(w, theta_np=W.random_parameters(11, pop, W.CNN_PARAMS, scale=0.1), members=members)


def test_cnn_tensor_core_path_is_deterministic():
    w = W.CFG3.with_(pop_size=8, batch=256)
    s = Solver(w)
    images, labels = W.image_batch(w.seed, 0, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    s.ask()
    a = s.rollout().clone(); b = s.rollout().clone()
    assert torch.equal(a, b) and s.sync_status() == 0
    s.close()


def test_cnn_rollout_needs_a_batch():
    from paper_2202_05008_b200 import EvoError
    s = Solver(W.CFG3.with_(pop_size=2, batch=8))
    s.ask()
    with pytest.raises(EvoError) as e:
        s.rollout()
    assert e.value.code == 2
    s.close()


@pytest.mark.parametrize("pop,batch", [(64, 256), (70, 48), (296, 16), (128, 100)])
def test_cnn_many_generations_stay_ok_and_deterministic(pop, batch):
    """The roles of the tensor-core kernels meet on mbarriers and progress counters; a rare ordering that made
    one of them wait for ever would show up as EVO_ERR_TIMEOUT (a bounded wait giving up) only after many
    launches.  150 generations per shape, the roll-out repeated now and then: same bits, status ok."""
    w = W.CFG3.with_(pop_size=pop, batch=batch)
    s = Solver(w)
    images, labels = W.image_batch(w.seed, 0, w.batch)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    fit = torch.empty(pop, dtype=torch.float32, device="cuda")
    for g in range(150):
        s.ask()
        s.rollout(fitness=fit)
        if g % 25 == 0:
            first = fit.clone()
            s.rollout(fitness=fit)
            assert torch.equal(first, fit)
        s.tell(fit)
    assert s.sync_status() == 0
    s.close()
