"""Pins of the seq2seq oracle (paper Section 3, "Seq2Seq Learning"): the LSTM encoder-decoder
against torch.nn.LSTM + Linear + cross_entropy (an independent library implementation), the
zero-parameter closed form, the bf16 reading against torch's own bfloat16 rounding, and the
generated queries against integer addition."""
import math

import numpy as np
import torch

import oracle

V = 12


def _torch_fitness(params, h, enc, dec, tgt, bf16=False):
    """The same network out of torch modules.  torch.nn.LSTM uses gate order (i, f, g, o) and two
    bias vectors; the second one is zero here."""
    p = torch.tensor(params, dtype=torch.float64)
    o = 0
    def take(n, shape):
        nonlocal o
        t = p[o:o + n].reshape(shape); o += n
        return t
    cells = []
    for _ in range(2):
        wx = take(4 * h * V, (4 * h, V)); wh = take(4 * h * h, (4 * h, h)); b = take(4 * h, (4 * h,))
        cells.append((wx, wh, b))
    ow = take(V * h, (V, h)); ob = take(V, (V,))
    assert o == p.numel()
    rnd = (lambda t: t.to(torch.float32).to(torch.bfloat16).to(torch.float64)) if bf16 else (lambda t: t)
    B = enc.shape[0]
    if not bf16:
        lstm_e = torch.nn.LSTM(V, h, batch_first=True).double()
        lstm_d = torch.nn.LSTM(V, h, batch_first=True).double()
        for mod, (wx, wh, b) in zip((lstm_e, lstm_d), cells):
            with torch.no_grad():
                mod.weight_ih_l0.copy_(wx); mod.weight_hh_l0.copy_(wh)
                mod.bias_ih_l0.copy_(b); mod.bias_hh_l0.zero_()
        x_e = torch.nn.functional.one_hot(torch.tensor(enc, dtype=torch.long), V).double()
        x_d = torch.nn.functional.one_hot(torch.tensor(dec, dtype=torch.long), V).double()
        with torch.no_grad():
            _, state = lstm_e(x_e)
            hs, _ = lstm_d(x_d, state)
            logits = hs @ ow.T + ob
    else:
        # step by step with LSTMCell-like algebra out of torch ops, rounding the operands of the
        # cell's contraction (Wh, Wx, b, h) and of the read-out (out.W, h) through torch's bfloat16
        hcur = torch.zeros(B, h, dtype=torch.float64); c = torch.zeros(B, h, dtype=torch.float64)
        outs = []
        for phase, toks in ((0, enc), (1, dec)):
            wx, wh, b = cells[phase]
            for t in range(toks.shape[1]):
                g = rnd(hcur) @ rnd(wh).T + rnd(wx)[:, torch.tensor(toks[:, t], dtype=torch.long)].T + rnd(b)
                i, f, gg, og = g.split(h, dim=1)
                c = torch.sigmoid(f) * c + torch.sigmoid(i) * torch.tanh(gg)
                hcur = torch.sigmoid(og) * torch.tanh(c)
                if phase == 1:
                    outs.append(rnd(hcur) @ rnd(ow).T + ob)
        logits = torch.stack(outs, dim=1)
    loss = torch.nn.functional.cross_entropy(logits.reshape(-1, V), torch.tensor(tgt, dtype=torch.long).reshape(-1))
    return -float(loss), logits.numpy()


def _params(h, scale, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(oracle.seq2seq_param_count(h)) * scale).astype(np.float32)


def test_param_count():
    assert oracle.seq2seq_param_count(128) == 2 * (512 * 12 + 512 * 128 + 512) + 12 * 128 + 12 == 145932
    assert oracle.seq2seq_param_count(4) == 2 * (16 * 12 + 16 * 4 + 16) + 48 + 12


def test_queries_spell_an_addition():
    for nd in (1, 3, 4):
        enc, dec, tgt = oracle.seq2seq_queries(7, 3, 500, nd)
        a = sum(enc[:, k].astype(np.int64) * 10 ** (nd - 1 - k) for k in range(nd))
        b = sum(enc[:, nd + 1 + k].astype(np.int64) * 10 ** (nd - 1 - k) for k in range(nd))
        s = sum(tgt[:, k].astype(np.int64) * 10 ** (nd - k) for k in range(nd + 1))
        assert np.all(enc[:, nd] == 10) and np.all(dec[:, 0] == 11)
        assert np.array_equal(a + b, s)
        assert np.array_equal(dec[:, 1:], tgt[:, :-1])             # teacher forcing: shifted answer
        assert enc.min() >= 0 and enc.max() <= 10 and tgt.max() <= 9
        assert len(set(zip(a.tolist(), b.tolist()))) > (5 if nd == 1 else 400)   # not a constant stream
        mid = (10 ** nd - 1) / 2                                   # uniform on 0 .. 10^nd - 1
        assert abs(a.mean() - mid) < 0.05 * 10 ** nd and abs(b.mean() - mid) < 0.05 * 10 ** nd
    e1, _, _ = oracle.seq2seq_queries(7, 3, 50, 3)
    e2, _, _ = oracle.seq2seq_queries(7, 4, 50, 3)
    e3, _, _ = oracle.seq2seq_queries(8, 3, 50, 3)
    assert not np.array_equal(e1, e2) and not np.array_equal(e1, e3)


def test_zero_parameters_give_log_vocab():
    enc, dec, tgt = oracle.seq2seq_queries(0, 0, 16, 3)
    f, acc = oracle.seq2seq_fitness(np.zeros(oracle.seq2seq_param_count(8), np.float32), 8, 3, enc, dec, tgt, True)
    assert abs(f + math.log(12)) < 1e-12
    # all logits tie at zero: the arg-max takes token 0, right exactly where the target digit is 0
    assert acc == np.mean(tgt == 0)


def test_matches_torch_lstm_unrounded():
    for h, nd, seed in ((8, 2, 1), (32, 3, 2), (128, 3, 3)):
        params = _params(h, 0.3, seed)
        enc, dec, tgt = oracle.seq2seq_queries(seed, 0, 12, nd)
        f, acc, logits = oracle.seq2seq_fitness(params, h, nd, enc, dec, tgt, False, want_logits=True)
        f_t, logits_t = _torch_fitness(params, h, enc, dec, tgt)
        assert np.max(np.abs(logits - logits_t)) < 1e-10
        assert abs(f - f_t) < 1e-12
        assert acc == np.mean(np.argmax(logits_t, axis=-1) == tgt)


def test_bf16_reading_matches_torch_bfloat16_rounding_points():
    h, nd = 32, 3
    params = _params(h, 0.3, 5)
    enc, dec, tgt = oracle.seq2seq_queries(5, 1, 10, nd)
    f, _, logits = oracle.seq2seq_fitness(params, h, nd, enc, dec, tgt, True, want_logits=True)
    f_t, logits_t = _torch_fitness(params, h, enc, dec, tgt, bf16=True)
    assert np.max(np.abs(logits - logits_t)) < 1e-10 and abs(f - f_t) < 1e-12
    f_exact, _ = oracle.seq2seq_fitness(params, h, nd, enc, dec, tgt, False)
    assert 0 < abs(f - f_exact) < 0.05                       # the rounding is there, and small


def test_forget_gate_carries_the_cell_state():
    """Saturated gates: i = 1, f = 0, o = 1 (biases +-40), cell input from the token only.  Then
    c_t = tanh(Wx_g[token_t]) and h_t = tanh(c_t) whatever came before: a hand-computable case."""
    h, nd = 2, 1
    n = oracle.seq2seq_param_count(h)
    p = np.zeros(n, np.float32)
    # decoder cell: offsets after the encoder block
    enc_block = 4 * h * V + 4 * h * h + 4 * h
    dWx = p[enc_block:enc_block + 4 * h * V].reshape(4 * h, V)
    db = p[enc_block + 4 * h * V + 4 * h * h:enc_block + 4 * h * V + 4 * h * h + 4 * h]
    db[0:h] = 40.0; db[h:2 * h] = -40.0; db[3 * h:4 * h] = 40.0
    dWx[2 * h + 0, :] = np.linspace(-1, 1, V); dWx[2 * h + 1, :] = 0.5
    oW = p[n - V - V * h:n - V].reshape(V, h)
    oW[3, 0] = 2.0; oW[7, 1] = -1.0
    enc, dec, tgt = oracle.seq2seq_queries(2, 0, 6, nd)
    f, _, logits = oracle.seq2seq_fitness(p, h, nd, enc, dec, tgt, False, want_logits=True)
    for i in range(6):
        for t in range(nd + 1):
            tok = dec[i, t]
            h0 = math.tanh(math.tanh(np.linspace(-1, 1, V).astype(np.float32)[tok]))
            h1 = math.tanh(math.tanh(0.5))
            want = np.zeros(V); want[3] = 2.0 * h0; want[7] = -1.0 * h1
            assert np.max(np.abs(logits[i, t] - want)) < 1e-12
