"""Synthetic workloads: the five configurations and the seeded input generators.

This module contains no arithmetic of the method itself.  It describes the shapes (population,
network, task, horizon) and produces the *inputs* the method does not draw for itself: image
batches and labels for the supervised task and the N(0,1) fitness vector of the update sweep.
The MNIST-shaped batches stand in for MNIST, which the paper's supervised example uses.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple

import numpy as np

NOISE_STORED, NOISE_REGENERATED = 0, 1
POLICY_NONE, POLICY_MLP, POLICY_CNN_28, POLICY_LSTM_SEQ2SEQ = 0, 1, 2, 3
TASK_NONE, TASK_CARTPOLE, TASK_TANH_LINEAR, TASK_SUPERVISED, TASK_SEQ2SEQ_ADD, TASK_PAINT = 0, 1, 2, 3, 4, 5
OPT_ADAM, OPT_CLIPUP = 0, 1
SIGMA_CONSTANT, SIGMA_PGPE = 0, 1

CNN_PARAMS = 5994


@dataclass(frozen=True)
class Workload:
    name: str
    pop_size: int
    param_dim: int
    seed: int
    sigma: float = 0.1
    lr: float = 0.01
    noise_mode: int = NOISE_STORED
    policy_kind: int = POLICY_NONE
    layer_sizes: Tuple[int, ...] = ()
    action_scale: float = 1.0
    task_kind: int = TASK_NONE
    episodes: int = 1
    horizon: int = 1
    batch: int = 0
    generations: int = 1
    # cart-pole: cart mass, pole mass, pole half length, gravity, dt, initial range; seq2seq: digits
    task_param: Tuple[float, ...] = field(default_factory=tuple)
    optimizer: int = OPT_ADAM
    clipup_momentum: float = 0.0          # 0 = library default (0.9)
    clipup_max_speed: float = 0.0         # 0 = library default (2 lr)
    sigma_mode: int = SIGMA_CONSTANT
    sigma_lr: float = 0.0                 # 0 = library default (0.1)
    sigma_max_change: float = 0.0         # 0 = library default (0.2)

    @property
    def env_steps_per_generation(self) -> int:
        if self.task_kind in (TASK_SUPERVISED, TASK_SEQ2SEQ_ADD):
            return self.pop_size * self.batch
        if self.task_kind == TASK_PAINT:
            return self.pop_size                 # one painted canvas per member
        if self.task_kind == TASK_NONE:
            return 0
        return self.pop_size * self.episodes * self.horizon

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def mlp_param_count(sizes) -> int:
    return sum(a * b + b for a, b in zip(sizes[:-1], sizes[1:]))


def _cartpole(init_range):
    return (1.0, 0.1, 0.5, 9.8, 0.01, init_range)


CFG1 = Workload("cfg1_cartpole_pop16", 16, 385, seed=0, policy_kind=POLICY_MLP,
                layer_sizes=(5, 16, 16, 1), action_scale=10.0, task_kind=TASK_CARTPOLE,
                episodes=1, horizon=200, generations=1, task_param=_cartpole(0.05))
CFG2 = Workload("cfg2_cartpole_pop256", 256, 4609, seed=0, policy_kind=POLICY_MLP,
                layer_sizes=(5, 64, 64, 1), action_scale=10.0, task_kind=TASK_CARTPOLE,
                episodes=16, horizon=1000, generations=100, task_param=_cartpole(0.2))
CFG3 = Workload("cfg3_cnn_pop64", 64, CNN_PARAMS, seed=1, policy_kind=POLICY_CNN_28,
                task_kind=TASK_SUPERVISED, batch=1024, generations=50)
CFG4 = Workload("cfg4_tanh_linear_pop4096", 4096, 21256, seed=2, policy_kind=POLICY_MLP,
                layer_sizes=(28, 128, 128, 8), action_scale=1.0, task_kind=TASK_TANH_LINEAR,
                episodes=4, horizon=1000, generations=20)
CFG5 = Workload("cfg5_update_sweep_pop16384", 16384, 1 << 20, seed=3, sigma=0.02,
                generations=1)



def seq2seq_param_count(h: int) -> int:
    return 2 * (4 * h * 12 + 4 * h * h + 4 * h) + 12 * h + 12


# the paper's seq2seq example (Section 3): LSTM encoder-decoder, 3-digit addition, a network of
# "hundreds of thousands of parameters" -> hidden width 128 gives 145,932
SEQ2SEQ = Workload("seq2seq_add_lstm128_pop1024", 1024, seq2seq_param_count(128), seed=4,
                   policy_kind=POLICY_LSTM_SEQ2SEQ, layer_sizes=(128,), task_kind=TASK_SEQ2SEQ_ADD,
                   batch=128, generations=20, task_param=(3.0,))

# the paper's painting example (Section 3): a canvas of semi-transparent triangles fitted to an
# image; task parameters = canvas width, height, background grey level
PAINT = Workload("paint_64_triangles_128x128_pop1024", 1024, 10 * 64, seed=5, sigma=0.1, lr=0.02,
                 task_kind=TASK_PAINT, generations=20, task_param=(128.0, 128.0, 0.0))


def paint_target(seed: int, width: int, height: int) -> np.ndarray:
    """Synthetic target image [H][W][3] fp32 in [0,1]: a few soft colour blobs and one hard-edged
    bar on a dark ground (stands in for the photographs the paper's example fits)."""
    rng = np.random.default_rng([seed, 0x7061696E74])
    y, x = np.meshgrid((np.arange(height) + 0.5) / height, (np.arange(width) + 0.5) / width, indexing="ij")
    img = np.full((height, width, 3), 0.05, np.float64)
    for _ in range(6):
        cx, cy, rad = rng.random(), rng.random(), 0.08 + 0.25 * rng.random()
        colour = rng.random(3)
        blob = np.exp(-((x - cx) ** 2 + (y - cy) ** 2) / (2 * rad * rad))
        img += blob[:, :, None] * colour[None, None, :] * 0.6
    x0, x1 = sorted(rng.random(2)); y0 = rng.random() * 0.8
    bar = (x >= x0) & (x <= x1) & (y >= y0) & (y <= y0 + 0.1)
    img[bar] = rng.random(3)
    return np.clip(img, 0.0, 1.0).astype(np.float32)


CONFIGS = {"cfg1": CFG1, "cfg2": CFG2, "cfg3": CFG3, "cfg4": CFG4, "cfg5": CFG5, "seq2seq": SEQ2SEQ, "paint": PAINT}

assert mlp_param_count(CFG1.layer_sizes) == CFG1.param_dim
assert mlp_param_count(CFG2.layer_sizes) == CFG2.param_dim
assert mlp_param_count(CFG4.layer_sizes) == CFG4.param_dim


def image_batch(seed: int, generation: int, batch: int):
    """Uniform [0,1) fp32 images [batch][28][28] and uniform labels {0..9} (int32)."""
    rng = np.random.default_rng([seed, generation, 0x696D67])
    images = rng.random((batch, 28, 28), dtype=np.float32)
    labels = rng.integers(0, 10, size=batch).astype(np.int32)
    return images, labels


def synthetic_fitness(seed: int, generation: int, pop_size: int) -> np.ndarray:
    """N(0,1) fitness, fp32, for the update sweep (no task is rolled out there)."""
    rng = np.random.default_rng([seed, generation, 0x666974])
    return rng.standard_normal(pop_size).astype(np.float32)


def random_parameters(seed: int, rows: int, dim: int, scale: float = 0.5) -> np.ndarray:
    """A dense [rows][dim] fp32 parameter matrix for teacher-forced rollout checks."""
    rng = np.random.default_rng([seed, 0x706172])
    return (rng.standard_normal((rows, dim)) * scale).astype(np.float32)
