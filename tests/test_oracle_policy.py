"""Pins for the oracle's policies: library routines, hand cases."""
import math

import numpy as np
import torch
import torch.nn.functional as F

import oracle


def test_mlp_param_counts_of_the_three_shapes():
    assert oracle.mlp_param_count([5, 16, 16, 1]) == 385
    assert oracle.mlp_param_count([5, 64, 64, 1]) == 4609
    assert oracle.mlp_param_count([28, 128, 128, 8]) == 21256


def test_mlp_matches_numpy_matmul():
    rng = np.random.default_rng(0)
    sizes = [5, 7, 3, 2]
    params = rng.standard_normal(oracle.mlp_param_count(sizes))
    x = rng.standard_normal(5)
    h, off = x, 0
    for n_in, n_out in zip(sizes[:-1], sizes[1:]):
        W = params[off:off + n_in * n_out].reshape(n_out, n_in); off += n_in * n_out
        b = params[off:off + n_out]; off += n_out
        h = np.tanh(W @ h + b)
    got = oracle.mlp_forward(params, sizes, x, action_scale=10.0)
    assert np.abs(got - 10.0 * h).max() < 1e-13


def test_mlp_not_transposed():
    # single layer 2 -> 1 with W = [1, 0]: output depends on x[0] only
    params = np.array([1.0, 0.0, 0.0])
    assert abs(oracle.mlp_forward(params, [2, 1], [0.5, 9.0])[0] - math.tanh(0.5)) < 1e-15
    # 1 -> 2 with W = [[2],[3]], b = [0.1, -0.1]
    params = np.array([2.0, 3.0, 0.1, -0.1])
    got = oracle.mlp_forward(params, [1, 2], [0.25])
    assert np.abs(got - np.tanh([0.6, 0.65])).max() < 1e-15


def _torch_cnn(params, images, bf16):
    p = torch.tensor(params, dtype=torch.float32)
    def op(t):
        return t.to(torch.bfloat16).to(torch.float64) if bf16 else t.to(torch.float64)
    w1 = p[0:200].reshape(8, 1, 5, 5); b1 = p[200:208]
    w2 = p[208:3408].reshape(16, 8, 5, 5); b2 = p[3408:3424]
    wf = p[3424:5984].reshape(10, 256); bf = p[5984:5994]
    x = torch.tensor(images, dtype=torch.float32).reshape(-1, 1, 28, 28)
    h = F.conv2d(op(x), op(w1)) + b1.double().view(1, -1, 1, 1)
    h = F.max_pool2d(F.relu(h), 2)
    h = F.conv2d(op(h.float()), op(w2)) + b2.double().view(1, -1, 1, 1)
    h = F.max_pool2d(F.relu(h), 2)
    return op(h.float()).reshape(-1, 256) @ op(wf).T + bf.double()


def test_cnn_matches_torch_layers():
    rng = np.random.default_rng(1)
    params = (rng.standard_normal(5994) * 0.1).astype(np.float32)
    images = rng.random((6, 28, 28), dtype=np.float32)
    labels = rng.integers(0, 10, size=6).astype(np.int32)
    for bf16 in (False, True):
        logits = _torch_cnn(params, images, bf16)
        for i in range(6):
            got = oracle.cnn_logits(params, images[i], bf16)
            assert np.abs(got - logits[i].numpy()).max() < (2e-2 if bf16 else 1e-5)
        want = -F.cross_entropy(logits, torch.tensor(labels, dtype=torch.long)).item()
        got = oracle.cnn_fitness(params, images, labels, bf16)
        assert abs(got - want) < (5e-3 if bf16 else 1e-6)


def test_cnn_zero_parameters_gives_minus_ln10():
    images = np.random.default_rng(2).random((5, 28, 28), dtype=np.float32)
    labels = np.array([0, 3, 9, 4, 4], dtype=np.int32)
    got = oracle.cnn_fitness(np.zeros(5994, dtype=np.float32), images, labels, True)
    assert abs(got + math.log(10.0)) < 1e-15


def test_cnn_single_path_by_hand():
    # one conv1 tap, one conv2 tap, one fc weight: logit 3 = image[2,3] (through two pools)
    params = np.zeros(5994, dtype=np.float32)
    params[0 * 25 + 2 * 5 + 3] = 1.0                       # conv1 filter 0, tap (2,3)
    params[208 + (5 * 8 + 0) * 25 + 1 * 5 + 1] = 2.0       # conv2 filter 5 <- channel 0, tap (1,1)
    params[3424 + 3 * 256 + 5 * 16 + 0 * 4 + 0] = 0.5      # fc class 3 <- (channel 5, 0, 0)
    image = np.zeros((28, 28), dtype=np.float32)
    # pool2(0,0) of filter 5 covers conv2 outputs (0..1, 0..1) <- pool1 (1..2, 1..2)
    # <- conv1 outputs (2..5, 2..5) <- image rows 4..7, cols 5..8
    image[4:8, 5:9] = np.array([[.1, .2, .3, .1], [.2, .9, .3, .1], [.1, .1, .1, .1], [.1, .1, .1, .7]])
    logits = oracle.cnn_logits(params, image, False)
    assert abs(logits[3] - 0.5 * 2.0 * 0.9) < 1e-6
    assert all(abs(logits[o]) < 1e-12 for o in range(10) if o != 3)


def test_bf16_rounding_ties_to_even():
    assert oracle.bf16_round(1.0) == 1.0
    assert oracle.bf16_round(1.0 + 2.0**-8) == 1.0                 # tie -> even mantissa
    assert oracle.bf16_round(1.0 + 3 * 2.0**-8) == 1.0 + 2.0**-6   # tie -> even (up)
    assert oracle.bf16_round(1.0 + 2.0**-8 + 2.0**-20) == 1.0 + 2.0**-7
    x = np.random.default_rng(3).standard_normal(1000).astype(np.float32)
    want = torch.tensor(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.bf16_round(v) for v in x], dtype=np.float32)
    assert (got == want).all()
