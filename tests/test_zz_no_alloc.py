"""The allocation-free gradient entry point against the regular tell path and the CPU oracle.

Some hosts of this library may not allocate device memory once they are running (a service that
hands out all GPU memory at boot, a plug-in under a framework that owns the allocator), so they
cannot give evo_create a workspace.  evo_es_gradient_static serves them with a fixed scratch array
inside the library.  Here its result is compared, through the C-ABI, with the gradient that
evo_tell computes from the same rank weights and noise and with the oracle's gradient of the same
inputs, on two calls in a row (the second call finds the scratch as the first left it).  This file sorts last so that a run stopping at the first
failure has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err
from paper_2202_05008_b200 import Solver, load_library, workloads as W
from paper_2202_05008_b200.binding import es_gradient_static, EvoError, STATIC_SCRATCH_BYTES

pytestmark = pytest.mark.gpu

TOL = 1e-5          # the bound the other tell tests use for the gradient


def _reference(w, generation_count=1):
    """(u, eps view, g) from the regular path after `generation_count` tells."""
    s = Solver(w)
    for g in range(generation_count):
        s.ask()
        s.tell(torch.tensor(W.synthetic_fitness(w.seed, g, w.pop_size), device="cuda"))
    assert s.sync_status() == 0
    _, u = s.ranks()
    return s, u.clone(), s.eps(), s.gradient().clone()


@pytest.mark.parametrize("P,D", [(256, 4609), (4096, 21256), (34, 7)])
def test_static_gradient_matches_tell_twice_in_a_row(P, D):
    w = W.Workload("noalloc", P, D, seed=P + D, sigma=0.1)
    s1, u1, eps1, g1 = _reference(w, 1)
    w2 = w.with_(seed=w.seed + 1)
    s2, u2, eps2, g2 = _reference(w2, 2)
    out = torch.empty(D, dtype=torch.float32, device="cuda")
    got1 = es_gradient_static(u1, eps1, w.sigma, out=out).clone()
    got2 = es_gradient_static(u2, eps2, w.sigma, out=out).clone()   # scratch holds call 1's sums
    torch.cuda.synchronize()
    assert rel_err(got1.cpu().numpy(), g1.cpu().numpy()) < TOL
    assert rel_err(got2.cpu().numpy(), g2.cpu().numpy()) < TOL
    # and against the CPU oracle directly (not only against another CUDA path)
    sigma32 = float(np.float32(w.sigma))
    for got, u, eps in ((got1, u1, eps1), (got2, u2, eps2)):
        want = oracle.gradient(u.cpu().numpy(), np.ascontiguousarray(eps.cpu().numpy()), sigma32)
        assert rel_err(got.cpu().numpy(), want) < TOL
    assert not torch.equal(got1, got2)
    # and once more with the first inputs: identical to the first answer
    got3 = es_gradient_static(u1, eps1, w.sigma, out=out)
    assert torch.equal(got3, got1)
    s1.close(); s2.close()


def test_static_gradient_rejects_sizes_beyond_the_fixed_scratch():
    lib = load_library()
    limit = STATIC_SCRATCH_BYTES // 8
    u = torch.zeros(2, device="cuda")
    eps = torch.zeros(1, 64, device="cuda")
    g = torch.zeros(64, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    # the size check comes before any pointer is used
    assert lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), 2, limit + 1, limit + 1, 0.1,
                                      g.data_ptr(), st) == 3
    # a parameter count whose rounding up to 32 would wrap a 32-bit integer is still "too large"
    assert lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), 2, 0xFFFFFFF0, 0xFFFFFFF0, 0.1,
                                      g.data_ptr(), st) == 3
    assert lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), 3, 64, 64, 0.1, g.data_ptr(), st) == 1
    assert lib.evo_es_gradient_static(None, eps.data_ptr(), 2, 64, 64, 0.1, g.data_ptr(), st) == 1
    assert lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), 2, 64, 32, 0.1, g.data_ptr(), st) == 1
    assert lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), 2, 64, 64, 0.1, g.data_ptr(), st) == 0
    torch.cuda.synchronize()
