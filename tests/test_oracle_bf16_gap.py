"""How far the bf16 reading of the two tensor-core policies moves the fitness.

The oracle has two modes for the CNN and the seq2seq network: operands of the contractions rounded
to bf16 (the reading "fp32 master, bf16 tensor-core forward"), and plain fp64 with nothing rounded
(pinned to torch's conv2d / nn.LSTM elsewhere).  The GPU kernels are compared with BOTH; the
looser bound used against the unrounded mode is the one pinned here, between the two oracle
modes, so it does not depend on any kernel.
"""
import numpy as np

import oracle
from paper_2202_05008_b200 import workloads as W

# |fitness(bf16 operands) - fitness(unrounded)| relative to max(|fitness|, 1); the GPU tests allow
# this much plus their own 1e-3 against the unrounded oracle.
BF16_GAP = 1e-3


def _gap(a, b):
    return abs(a - b) / max(abs(b), 1.0)


def test_cnn_bf16_reading_stays_within_the_gap_bound():
    w = W.CFG3
    images, labels = W.image_batch(w.seed, 0, 128)
    th, _ = oracle.ask(w.seed, 0, 8, w.param_dim, np.zeros(w.param_dim, np.float32), w.sigma)
    rows = list(th[:4]) + list(W.random_parameters(9, 3, W.CNN_PARAMS, scale=0.1))
    gaps = [_gap(oracle.cnn_fitness(r, images, labels, True), oracle.cnn_fitness(r, images, labels, False))
            for r in rows]
    assert max(gaps) < BF16_GAP
    assert max(gaps) > 1e-7                      # the two modes really differ


def test_seq2seq_bf16_reading_stays_within_the_gap_bound():
    w = W.SEQ2SEQ
    enc, dec, tgt = oracle.seq2seq_queries(w.seed, 0, 32, 3)
    th, _ = oracle.ask(w.seed, 0, 4, w.param_dim, np.zeros(w.param_dim, np.float32), w.sigma)
    rows = list(th[:2]) + list(W.random_parameters(3, 2, w.param_dim, scale=0.3))
    gaps = [_gap(oracle.seq2seq_fitness(r, 128, 3, enc, dec, tgt, True)[0],
                 oracle.seq2seq_fitness(r, 128, 3, enc, dec, tgt, False)[0]) for r in rows]
    assert max(gaps) < BF16_GAP
    assert max(gaps) > 1e-8
