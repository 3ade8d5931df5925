"""Edge cases of the C-ABI on a device: argument errors, minimal and odd sizes."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from helpers import rel_err, oracle_fitness
from paper_2202_05008_b200 import Solver, EvoError, load_library, workloads as W
from paper_2202_05008_b200.binding import make_config, ROLLOUT_TILED, ROLLOUT_GENERIC

pytestmark = pytest.mark.gpu


def test_create_rejects_small_workspace_and_unsupported_tiled_request():
    lib = load_library()
    cfg = make_config(W.CFG1)
    n = C.c_size_t()
    assert lib.evo_workspace_bytes(C.byref(cfg), C.byref(n)) == 0
    ws = torch.empty(n.value + 256, dtype=torch.uint8, device="cuda")
    ptr = (ws.data_ptr() + 255) // 256 * 256
    h = C.c_void_p()
    assert lib.evo_create(C.byref(cfg), ptr, n.value - 1, None, C.byref(h)) == 3      # workspace too small
    assert lib.evo_create(C.byref(cfg), ptr + 4, n.value, None, C.byref(h)) == 1      # misaligned
    # a shape no compiled fast kernel covers (wider than all of them): AUTO falls back to the generic
    # kernel, TILED is refused at rollout
    sizes = (5, 200, 12, 1)
    w = W.CFG1.with_(layer_sizes=sizes, param_dim=W.mlp_param_count(sizes), horizon=10)
    s = Solver(w, rollout_kernel=ROLLOUT_TILED)
    s.ask()
    with pytest.raises(EvoError) as e:
        s.rollout()
    assert e.value.code == 7
    s.close()
    torch.cuda.synchronize()


def test_rollout_argument_errors():
    lib = load_library()
    s = Solver(W.CFG1.with_(horizon=10))
    fit = torch.zeros(16, device="cuda")
    assert lib.evo_rollout(s._h, None, fit.data_ptr(), None) == 2                     # no ask yet
    s.ask()
    assert lib.evo_rollout(s._h, None, None, None) == 1                               # no fitness buffer
    theta = s.padded_rows(17)
    assert lib.evo_rollout(s._h, theta.data_ptr() + 4, fit.data_ptr(), None) == 1     # misaligned matrix
    trace = torch.zeros(16 * 10 * 4, device="cuda")
    assert lib.evo_rollout(s._h, None, fit.data_ptr(), trace.data_ptr()) == 1         # trace_steps is 0
    assert lib.evo_rollout(s._h, None, fit.data_ptr(), None) == 0
    assert s.sync_status() == 0
    s.close()
    # the trace is written with 128-bit stores: a pointer that is only 4-byte aligned is refused
    s = Solver(W.CFG1.with_(horizon=10), trace_steps=10)
    s.ask()
    trace = torch.zeros(16 * 10 * 4 + 4, device="cuda")
    assert lib.evo_rollout(s._h, None, fit.data_ptr(), trace.data_ptr() + 4) == 1
    assert lib.evo_rollout(s._h, None, fit.data_ptr(), trace.data_ptr()) == 0
    assert s.sync_status() == 0
    s.close()


def _with_batch(s, w):
    if w.task_kind == W.TASK_SUPERVISED:
        images, labels = W.image_batch(w.seed, 0, w.batch)
        s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    return s


@pytest.mark.parametrize("w", [W.CFG1.with_(horizon=5), W.CFG2.with_(pop_size=4, horizon=5),
                               W.CFG4.with_(pop_size=4, horizon=5), W.CFG3.with_(pop_size=6, batch=40)])
def test_a_device_wait_that_runs_out_raises_timeout_and_leaves_the_solver_usable(w):
    """The failure path of the bounded waits, made to happen without disturbing the device: with
    EVO_DEBUG_DROP_COMPLETION the roll-out blocks never start the copy they wait for, and with a
    limit of 2^16 clocks the wait gives up after ~30 us.  Every block must return by itself, raise
    EVO_ERR_TIMEOUT and report NaN; evo_sync_status must report the condition once and clear it; a
    tell on that fitness must skip the update (NaN fitness)."""
    from paper_2202_05008_b200.binding import DEBUG_DROP_COMPLETION
    s = _with_batch(Solver(w, wait_cycles_log2=16, debug_flags=DEBUG_DROP_COMPLETION), w)
    s.ask()
    fit = s.rollout()
    assert s.sync_status() == 6                        # EVO_ERR_TIMEOUT, reported ...
    assert s.sync_status() == 0                        # ... once
    assert bool(torch.isnan(fit).all())
    c0 = s.center().clone()
    s.tell(fit)
    assert s.sync_status() == 5                        # NaN fitness: update skipped
    assert torch.equal(s.center(), c0) and s.counters() == (1, 0)
    s.close()
    # the same configuration without the flag runs normally afterwards on the same device
    s = _with_batch(Solver(w, wait_cycles_log2=22), w)
    s.ask()
    fit = s.rollout()
    assert s.sync_status() == 0 and bool(torch.isfinite(fit).all())
    s.close()


@pytest.mark.parametrize("kernel", [ROLLOUT_GENERIC, ROLLOUT_TILED])
def test_smallest_population_single_step_single_episode(kernel):
    w = W.CFG1.with_(pop_size=2, horizon=1, episodes=1)
    s = Solver(w, trace_steps=1, rollout_kernel=kernel)
    th = s.ask().cpu().numpy()
    trace = torch.zeros(2, 1, 1, 4, device="cuda")
    fit = s.rollout(trace=trace).cpu().numpy()
    fit_o, tr_o = oracle_fitness(w, th, 0, 1, want_trace=True)
    assert rel_err(fit, fit_o, floor=1.0) < 1e-3
    assert np.abs(trace.cpu().numpy()[0, 0, 0] - tr_o[0][0, 0]).max() < 1e-5
    s.tell(torch.tensor(fit, device="cuda"))
    rank, u = (x.cpu().numpy() for x in s.ranks())
    assert sorted(rank.tolist()) == [0, 1] and sorted(u.tolist()) == [-0.5, 0.5]
    assert s.sync_status() == 0
    s.close()


def test_many_episodes_on_the_small_network():
    w = W.CFG1.with_(episodes=100, horizon=20, pop_size=4)
    s = Solver(w)
    th = s.ask().cpu().numpy()
    fit = s.rollout().cpu().numpy()
    fit_o, _ = oracle_fitness(w, th, 0, 20)
    assert rel_err(fit, fit_o, floor=1.0) < 1e-3
    s.close()


def test_cnn_single_image_batch():
    w = W.CFG3.with_(pop_size=2, batch=1)
    s = Solver(w)
    images, labels = W.image_batch(w.seed, 0, 1)
    s.set_batch(torch.tensor(images, device="cuda"), torch.tensor(labels, device="cuda"))
    th = W.random_parameters(9, 2, W.CNN_PARAMS, scale=0.1)
    arg = s.padded_rows(2); arg[:, :W.CNN_PARAMS] = torch.tensor(th, device="cuda")
    fit = s.rollout(arg).cpu().numpy()
    want = np.array([oracle.cnn_fitness(th[m], images, labels, True) for m in range(2)])
    assert rel_err(fit, want, floor=1.0) < 1e-3 and s.sync_status() == 0
    s.close()


def test_fma_probe_reports_a_plausible_fp32_rate_and_rejects_bad_shapes():
    """The probe is bench.py's measurement aid (its own shared object beside bench.py)."""
    import ctypes as C
    import bench
    rate = bench.fma_probe(iters=1 << 12, repeats=2)
    assert 5.0 < rate < 200.0                          # TFLOP/s; nominal is about 74
    lib = bench._probe
    sink = torch.empty(1024, dtype=torch.float32, device="cuda")
    flops = C.c_uint64()
    assert lib.bench_fma_probe(sink.data_ptr(), 1, 48, 8, None, C.byref(flops)) == 1      # not a warp multiple
    assert lib.bench_fma_probe(None, 1, 32, 8, None, C.byref(flops)) == 1
    assert lib.bench_fma_probe(sink.data_ptr(), 1, 1024, 8, None, C.byref(flops)) == 0
    torch.cuda.synchronize()
    assert flops.value == 2 * 16 * 8 * 1024


@pytest.mark.parametrize("w", [W.CFG1.with_(pop_size=32), W.CFG3.with_(pop_size=70, batch=48),
                               W.CFG4.with_(pop_size=8, horizon=20)])
def test_graph_replay_of_a_generation_matches_plain_calls(w):
    """ask -> rollout -> tell captured once and replayed must walk through the same generations
    (same noise, same episode seeds, same centre) as the three calls made one by one.  The kernels of a
    generation are programmatic dependents of one another; the capture must keep those edges."""
    plain = _with_batch(Solver(w), w)
    for _ in range(4):
        plain.ask()
        plain.tell(plain.rollout())
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = _with_batch(Solver(w, stream=side), w)
        fit = torch.empty(w.pop_size, device="cuda")
        g.ask(); g.tell(g.rollout(fitness=fit))                  # generation 0 by hand (also warms up)
        graph = g.capture_generation(fit)                         # capturing does not run anything
        for _ in range(3):
            graph.replay()
        side.synchronize()
    assert g.counters() == plain.counters() == (4, 4)
    assert torch.equal(g.center(), plain.center())
    assert g.sync_status() == 0
    with pytest.raises(ValueError):
        plain.capture_generation(fit)                             # default stream cannot be captured
