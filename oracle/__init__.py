"""CPU oracle for one evolution-strategy generation -- TEST INFRASTRUCTURE ONLY.

A thin ctypes view of ``liboracle.so`` (plain C, fp64, single-threaded; see
``oracle.h``).  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this package; the CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = ["rng.c", "solver.c", "policy.c", "tasks.c", "seq2seq.c", "paint.c"]
_LIB_PATH = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved)."""
    srcs = [os.path.join(_HERE, s) for s in _SRC] + [os.path.join(_HERE, "oracle.h")]
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in srcs)
    if stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-o", _LIB_PATH] + [os.path.join(_HERE, s) for s in _SRC] + ["-lm"]
        subprocess.run(cmd, check=True)
    return _LIB_PATH


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


class CartpoleParams(C.Structure):
    _fields_ = [("cart_mass", C.c_double), ("pole_mass", C.c_double),
                ("pole_half_length", C.c_double), ("gravity", C.c_double),
                ("dt", C.c_double), ("integrator", C.c_int)]


def cartpole_params(cart_mass=1.0, pole_mass=0.1, pole_half_length=0.5, gravity=9.8,
                    dt=0.01, integrator=0) -> CartpoleParams:
    return CartpoleParams(cart_mass, pole_mass, pole_half_length, gravity, dt, integrator)


_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)
_u32p = C.POINTER(C.c_uint32)
_i32p = C.POINTER(C.c_int32)


def _declare(L):
    L.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
    L.oracle_stream_words.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, _u32p]
    L.oracle_u_open.argtypes = [C.c_uint32]; L.oracle_u_open.restype = C.c_float
    L.oracle_u_half.argtypes = [C.c_uint32]; L.oracle_u_half.restype = C.c_float
    L.oracle_ln_f32.argtypes = [C.c_float]; L.oracle_ln_f32.restype = C.c_float
    L.oracle_cossin_2pi_f32.argtypes = [C.c_float, _f32p, _f32p]
    L.oracle_normal4.argtypes = [_u32p, _f32p]
    L.oracle_eps_row.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, _f32p]
    L.oracle_ask.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, _f32p, C.c_float, _f32p, _f32p]
    L.oracle_centered_rank.argtypes = [_f32p, C.c_uint32, _i32p, _f32p]
    L.oracle_centered_rank.restype = C.c_int
    L.oracle_gradient.argtypes = [_f32p, _f32p, C.c_uint32, C.c_uint32, C.c_double, _f64p]
    L.oracle_adam.argtypes = [_f64p, _f64p, _f64p, _f64p, C.c_uint32, C.c_uint32,
                              C.c_double, C.c_double, C.c_double, C.c_double]
    L.oracle_ask_sigma.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, _f32p, _f32p, _f32p, _f32p]
    L.oracle_gradient_sigma.argtypes = [_f32p, _f32p, C.c_uint32, C.c_uint32, _f64p, _f64p]
    L.oracle_sigma_gradient.argtypes = [_f32p, _f32p, C.c_uint32, C.c_uint32, _f64p, _f64p]
    L.oracle_sigma_update.argtypes = [_f64p, _f64p, C.c_uint32, C.c_double, C.c_double]
    L.oracle_clipup.argtypes = [_f64p, _f64p, _f64p, C.c_uint32, C.c_double, C.c_double, C.c_double]
    L.oracle_mlp_forward.argtypes = [_f64p, C.c_uint32, _u32p, _f64p, _f64p, C.c_double]
    L.oracle_mlp_param_count.argtypes = [C.c_uint32, _u32p]
    L.oracle_mlp_param_count.restype = C.c_uint32
    L.oracle_cnn_fitness.argtypes = [_f32p, _f32p, _i32p, C.c_uint32, C.c_int]
    L.oracle_cnn_fitness.restype = C.c_double
    L.oracle_paint_inside.argtypes = [_f32p, C.c_float, C.c_float]
    L.oracle_paint_inside.restype = C.c_int
    L.oracle_paint_render.argtypes = [_f32p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_double, _f64p]
    L.oracle_paint_fitness.argtypes = [_f32p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_double, _f32p, _f64p]
    L.oracle_paint_fitness.restype = C.c_double
    L.oracle_seq2seq_param_count.argtypes = [C.c_uint32]
    L.oracle_seq2seq_param_count.restype = C.c_uint32
    L.oracle_seq2seq_queries.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, _i32p, _i32p, _i32p]
    L.oracle_seq2seq_fitness.argtypes = [_f32p, C.c_uint32, C.c_uint32, C.c_uint32, _i32p, _i32p, _i32p,
                                         C.c_int, _f64p, _f64p]
    L.oracle_seq2seq_fitness.restype = C.c_double
    L.oracle_cnn_logits.argtypes = [_f32p, _f32p, C.c_int, _f64p]
    L.oracle_bf16_round.argtypes = [C.c_float]; L.oracle_bf16_round.restype = C.c_float
    L.oracle_cartpole_reset.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_float, _f32p]
    L.oracle_cartpole_step.argtypes = [C.POINTER(CartpoleParams), _f64p, C.c_double]
    L.oracle_cartpole_energy.argtypes = [C.POINTER(CartpoleParams), _f64p]
    L.oracle_cartpole_energy.restype = C.c_double
    L.oracle_cartpole_momentum.argtypes = [C.POINTER(CartpoleParams), _f64p]
    L.oracle_cartpole_momentum.restype = C.c_double
    L.oracle_rollout_cartpole.argtypes = [_f32p, C.c_uint32, _u32p, C.c_double,
                                          C.POINTER(CartpoleParams), C.c_float, C.c_uint64,
                                          C.c_uint32, C.c_uint32, C.c_uint32, _f64p]
    L.oracle_rollout_cartpole.restype = C.c_double
    L.oracle_tanh_linear_constants.argtypes = [C.c_uint64, _f32p, _f32p]
    L.oracle_tanh_linear_reset.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, _f32p]
    L.oracle_rollout_tanh_linear.argtypes = [_f32p, C.c_uint32, _u32p, C.c_double, _f32p, _f32p,
                                             C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, _f64p]
    L.oracle_rollout_tanh_linear.restype = C.c_double


def _p(a, t):
    return a.ctypes.data_as(t)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _sizes(sizes):
    return np.ascontiguousarray(sizes, dtype=np.uint32)


# ---- random numbers ---------------------------------------------------------------

def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy(); k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c, _u32p), _p(k, _u32p), _p(out, _u32p))
    return out


def stream_words(seed, stream, generation, row, item):
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_stream_words(seed, stream, generation, row, item, _p(out, _u32p))
    return out


def u_open(r): return float(lib().oracle_u_open(int(r)))
def u_half(r): return float(lib().oracle_u_half(int(r)))
def ln_f32(u): return float(lib().oracle_ln_f32(float(u)))


def cossin_2pi_f32(v):
    c = C.c_float(); s = C.c_float()
    lib().oracle_cossin_2pi_f32(float(v), C.byref(c), C.byref(s))
    return c.value, s.value


def normal4(r):
    rr = np.asarray(r, dtype=np.uint32).copy(); z = np.zeros(4, dtype=np.float32)
    lib().oracle_normal4(_p(rr, _u32p), _p(z, _f32p))
    return z


# ---- solver -----------------------------------------------------------------------

def eps_row(seed, generation, pair, D):
    eps = np.zeros(D, dtype=np.float32)
    lib().oracle_eps_row(seed, generation, pair, D, _p(eps, _f32p))
    return eps


def ask(seed, generation, P, D, center, sigma, want_eps=True):
    center = _f32(center)
    theta = np.zeros((P, D), dtype=np.float32)
    eps = np.zeros((P // 2, D), dtype=np.float32) if want_eps else None
    lib().oracle_ask(seed, generation, P, D, _p(center, _f32p), float(sigma), _p(theta, _f32p),
                     _p(eps, _f32p) if want_eps else None)
    return theta, eps


def centered_rank(fitness):
    f = _f32(fitness); P = f.shape[0]
    rank = np.zeros(P, dtype=np.int32); u = np.zeros(P, dtype=np.float32)
    bad = lib().oracle_centered_rank(_p(f, _f32p), P, _p(rank, _i32p), _p(u, _f32p))
    return rank, u, bool(bad)


def gradient(u, eps, sigma):
    u = _f32(u); eps = _f32(eps); H, D = eps.shape
    g = np.zeros(D, dtype=np.float64)
    lib().oracle_gradient(_p(u, _f32p), _p(eps, _f32p), 2 * H, D, float(sigma), _p(g, _f64p))
    return g


def adam(center, m, v, g, t, lr, beta1=0.9, beta2=0.999, adam_eps=1e-8):
    """Returns updated (center, m, v) as fp64 copies."""
    c = np.array(center, dtype=np.float64); mm = np.array(m, dtype=np.float64)
    vv = np.array(v, dtype=np.float64); gg = np.ascontiguousarray(g, dtype=np.float64)
    lib().oracle_adam(_p(c, _f64p), _p(mm, _f64p), _p(vv, _f64p), _p(gg, _f64p), c.shape[0], t,
                      lr, beta1, beta2, adam_eps)
    return c, mm, vv


def ask_sigma(seed, generation, P, D, center, sigma, want_eps=True):
    center = _f32(center); sigma = _f32(sigma)
    theta = np.zeros((P, D), dtype=np.float32)
    eps = np.zeros((P // 2, D), dtype=np.float32) if want_eps else None
    lib().oracle_ask_sigma(seed, generation, P, D, _p(center, _f32p), _p(sigma, _f32p), _p(theta, _f32p),
                           _p(eps, _f32p) if want_eps else None)
    return theta, eps


def gradient_sigma(u, eps, sigma):
    u = _f32(u); eps = _f32(eps); H, D = eps.shape
    sg = np.ascontiguousarray(sigma, dtype=np.float64); g = np.zeros(D, dtype=np.float64)
    lib().oracle_gradient_sigma(_p(u, _f32p), _p(eps, _f32p), 2 * H, D, _p(sg, _f64p), _p(g, _f64p))
    return g


def sigma_gradient(u, eps, sigma):
    u = _f32(u); eps = _f32(eps); H, D = eps.shape
    sg = np.ascontiguousarray(sigma, dtype=np.float64); gs = np.zeros(D, dtype=np.float64)
    lib().oracle_sigma_gradient(_p(u, _f32p), _p(eps, _f32p), 2 * H, D, _p(sg, _f64p), _p(gs, _f64p))
    return gs


def sigma_update(sigma, gs, lr_sigma, max_change):
    sg = np.array(sigma, dtype=np.float64); g = np.ascontiguousarray(gs, dtype=np.float64)
    lib().oracle_sigma_update(_p(sg, _f64p), _p(g, _f64p), sg.shape[0], float(lr_sigma), float(max_change))
    return sg


def clipup(center, velocity, g, lr, momentum, max_speed):
    c = np.array(center, dtype=np.float64); v = np.array(velocity, dtype=np.float64)
    gg = np.ascontiguousarray(g, dtype=np.float64)
    lib().oracle_clipup(_p(c, _f64p), _p(v, _f64p), _p(gg, _f64p), c.shape[0], float(lr), float(momentum),
                        float(max_speed))
    return c, v


# ---- policies ---------------------------------------------------------------------

def mlp_param_count(sizes):
    s = _sizes(sizes)
    return int(lib().oracle_mlp_param_count(len(s) - 1, _p(s, _u32p)))


def mlp_forward(params, sizes, x, action_scale=1.0):
    s = _sizes(sizes)
    p = np.ascontiguousarray(params, dtype=np.float64); xx = np.ascontiguousarray(x, dtype=np.float64)
    y = np.zeros(int(s[-1]), dtype=np.float64)
    lib().oracle_mlp_forward(_p(p, _f64p), len(s) - 1, _p(s, _u32p), _p(xx, _f64p), _p(y, _f64p),
                             float(action_scale))
    return y


def cnn_fitness(params, images, labels, bf16_operands=True):
    p = _f32(params); im = _f32(images); lb = np.ascontiguousarray(labels, dtype=np.int32)
    return float(lib().oracle_cnn_fitness(_p(p, _f32p), _p(im, _f32p), _p(lb, _i32p), im.shape[0],
                                          int(bool(bf16_operands))))


def cnn_logits(params, image, bf16_operands=True):
    p = _f32(params); im = _f32(image); out = np.zeros(10, dtype=np.float64)
    lib().oracle_cnn_logits(_p(p, _f32p), _p(im, _f32p), int(bool(bf16_operands)), _p(out, _f64p))
    return out


def bf16_round(x): return float(lib().oracle_bf16_round(float(x)))


def paint_inside(tri6, px, py):
    t = _f32(tri6)
    return bool(lib().oracle_paint_inside(_p(t, _f32p), float(px), float(py)))


def paint_render(params, W, H, background=0.0):
    """Canvas [H][W][3] (fp64) of the triangles in `params` ([N][10] raw numbers)."""
    p = _f32(params).reshape(-1)
    canvas = np.zeros((H, W, 3), np.float64)
    lib().oracle_paint_render(_p(p, _f32p), p.size // 10, W, H, float(background), _p(canvas, _f64p))
    return canvas


def paint_fitness(params, W, H, target, background=0.0):
    p = _f32(params).reshape(-1); t = _f32(target)
    assert t.shape == (H, W, 3)
    canvas = np.zeros((H, W, 3), np.float64)
    return float(lib().oracle_paint_fitness(_p(p, _f32p), p.size // 10, W, H, float(background),
                                            _p(t, _f32p), _p(canvas, _f64p)))


def seq2seq_param_count(h): return int(lib().oracle_seq2seq_param_count(int(h)))


def seq2seq_queries(seed, generation, B, nd):
    """(encoder tokens [B][2nd+1], decoder input tokens [B][nd+1], targets [B][nd+1]), int32."""
    enc = np.zeros((B, 2 * nd + 1), np.int32); dec = np.zeros((B, nd + 1), np.int32)
    tgt = np.zeros((B, nd + 1), np.int32)
    lib().oracle_seq2seq_queries(int(seed), int(generation), B, nd, _p(enc, _i32p), _p(dec, _i32p), _p(tgt, _i32p))
    return enc, dec, tgt


def seq2seq_fitness(params, h, nd, enc, dec, tgt, bf16_operands=True, want_logits=False):
    """(fitness, accuracy[, logits [B][nd+1][12]]) of one member's LSTM encoder-decoder."""
    p = _f32(params)
    assert p.size == seq2seq_param_count(h)
    enc = np.ascontiguousarray(enc, np.int32); dec = np.ascontiguousarray(dec, np.int32)
    tgt = np.ascontiguousarray(tgt, np.int32)
    B = enc.shape[0]
    acc = np.zeros(1, np.float64)
    logits = np.zeros((B, nd + 1, 12), np.float64) if want_logits else None
    f = float(lib().oracle_seq2seq_fitness(_p(p, _f32p), h, nd, B, _p(enc, _i32p), _p(dec, _i32p), _p(tgt, _i32p),
                                           int(bool(bf16_operands)), _p(acc, _f64p),
                                           _p(logits, _f64p) if want_logits else None))
    return (f, float(acc[0]), logits) if want_logits else (f, float(acc[0]))


# ---- tasks ------------------------------------------------------------------------

def cartpole_reset(seed, generation, episode, init_range):
    s0 = np.zeros(4, dtype=np.float32)
    lib().oracle_cartpole_reset(seed, generation, episode, float(init_range), _p(s0, _f32p))
    return s0


def cartpole_step(params: CartpoleParams, state, force):
    s = np.array(state, dtype=np.float64)
    lib().oracle_cartpole_step(C.byref(params), _p(s, _f64p), float(force))
    return s


def cartpole_energy(params, state):
    s = np.array(state, dtype=np.float64)
    return float(lib().oracle_cartpole_energy(C.byref(params), _p(s, _f64p)))


def cartpole_momentum(params, state):
    s = np.array(state, dtype=np.float64)
    return float(lib().oracle_cartpole_momentum(C.byref(params), _p(s, _f64p)))


def rollout_cartpole(theta_row, sizes, action_scale, params, init_range, seed, generation, E, T,
                     want_trace=False):
    th = _f32(theta_row); s = _sizes(sizes)
    trace = np.zeros((E, T, 4), dtype=np.float64) if want_trace else None
    fit = lib().oracle_rollout_cartpole(_p(th, _f32p), len(s) - 1, _p(s, _u32p), float(action_scale),
                                        C.byref(params), float(init_range), seed, generation, E, T,
                                        _p(trace, _f64p) if want_trace else None)
    return float(fit), trace


def tanh_linear_constants(seed):
    A = np.zeros((28, 28), dtype=np.float32); B = np.zeros((28, 8), dtype=np.float32)
    lib().oracle_tanh_linear_constants(seed, _p(A, _f32p), _p(B, _f32p))
    return A, B


def tanh_linear_reset(seed, generation, episode):
    x0 = np.zeros(28, dtype=np.float32)
    lib().oracle_tanh_linear_reset(seed, generation, episode, _p(x0, _f32p))
    return x0


def rollout_tanh_linear(theta_row, sizes, action_scale, A, B, seed, generation, E, T, want_trace=False):
    th = _f32(theta_row); s = _sizes(sizes); A = _f32(A); B = _f32(B)
    trace = np.zeros((E, T, 28), dtype=np.float64) if want_trace else None
    fit = lib().oracle_rollout_tanh_linear(_p(th, _f32p), len(s) - 1, _p(s, _u32p), float(action_scale),
                                           _p(A, _f32p), _p(B, _f32p), seed, generation, E, T,
                                           _p(trace, _f64p) if want_trace else None)
    return float(fit), trace
