"""Shared helpers of the GPU parity tests (comparison metrics, oracle drivers)."""
import numpy as np

import oracle
from paper_2202_05008_b200 import workloads as W


def rel_err(a, b, floor=None):
    """max_i |a_i - b_i| / max(|b_i|, floor); floor defaults to RMS(b)."""
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    if floor is None:
        floor = float(np.sqrt(np.mean(b * b))) or 1.0
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), floor)))


def oracle_fitness(w: W.Workload, theta_rows, generation, T=None, want_trace=False, consts=None):
    """Oracle rollouts of the given dense parameter rows; returns (fitness[rows], traces)."""
    T = w.horizon if T is None else T
    fits, traces = [], []
    for row in theta_rows:
        if w.task_kind == W.TASK_CARTPOLE:
            tp = w.task_param
            p = oracle.cartpole_params(tp[0], tp[1], tp[2], tp[3], tp[4])
            f, tr = oracle.rollout_cartpole(row, w.layer_sizes, w.action_scale, p, tp[5], w.seed,
                                            generation, w.episodes, T, want_trace)
        elif w.task_kind == W.TASK_TANH_LINEAR:
            A, B = consts if consts is not None else oracle.tanh_linear_constants(w.seed)
            f, tr = oracle.rollout_tanh_linear(row, w.layer_sizes, w.action_scale, A, B, w.seed,
                                               generation, w.episodes, T, want_trace)
        else:
            raise ValueError(w.task_kind)
        fits.append(f); traces.append(tr)
    return np.array(fits), traces


def cartpole_features(trace):
    """(x, x', sin, cos, theta') from raw (x, x', theta, theta') states."""
    t = np.asarray(trace, dtype=np.float64)
    return np.stack([t[..., 0], t[..., 1], np.sin(t[..., 2]), np.cos(t[..., 2]), t[..., 3]], axis=-1)
