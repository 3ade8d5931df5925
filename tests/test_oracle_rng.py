"""Pins for the oracle's random numbers: published vectors, exactness, libm, moments."""
import math
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kat_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


def test_philox_cxx26_engine_check_value():
    kv = dict(l.split() for l in open(os.path.join(GOLDEN, "philox_engine_check.txt"))
              if l.strip() and not l.startswith("#"))
    seed, index, want = int(kv["seed"]), int(kv["index"]), int(kv["value"])
    n = (index - 1) // 4
    out = oracle.philox4x32_10([n, 0, 0, 0], [seed, 0])
    assert int(out[(index - 1) % 4]) == want


def test_stream_words_is_philox_with_documented_counter_layout():
    seed = 0x123456789ABCDEF
    got = oracle.stream_words(seed, 3, 7, 11, 13)
    want = oracle.philox4x32_10([13, 11, 7, 3], [seed & 0xFFFFFFFF, seed >> 32])
    assert (got == want).all()


def test_uniforms_are_exact_and_in_range():
    for r in [0, 1, 255, 256, 0x80000000, 0xFFFFFF00, 0xFFFFFFFF, 0x12345678]:
        k = r >> 8
        assert oracle.u_half(r) == k / 2.0**24
        assert oracle.u_open(r) == (k + 1) / 2.0**24
    assert oracle.u_half(0xFFFFFFFF) < 1.0 and oracle.u_half(0) == 0.0
    assert oracle.u_open(0xFFFFFFFF) == 1.0 and oracle.u_open(0) > 0.0


def test_trig_coefficients_are_fp32_roundings_of_the_factorial_fractions():
    # bit patterns that both implementations type in for sin (to x^9) and cos (to x^10)
    fact = {2: 0x3F000000, 3: 0x3E2AAAAB, 4: 0x3D2AAAAB, 5: 0x3C088889, 6: 0x3AB60B61,
            7: 0x39500D01, 8: 0x37D00D01, 9: 0x3638EF1D, 10: 0x3493F27E}
    for n, bits in fact.items():
        assert np.float32(1.0) / np.float32(math.factorial(n)) == np.uint32(bits).view(np.float32)


def test_ln_polynomial_is_a_fit_of_the_log_series_remainder():
    # P(f) ~ (ln(1+f) - f + f^2/2) / f^3 on [sqrt(1/2)-1, sqrt(2)-1]: the stated coefficients must
    # reproduce that function (an independent check of the table, in fp64)
    bits = [0x3EAAAAA9, 0xBE800064, 0x3E4CD0A6, 0xBE2A6AA7, 0x3E116E25, 0xBE04D5F2, 0x3E022C8D, 0xBDA5EB80]
    c = np.array(bits, dtype=np.uint32).view(np.float32).astype(np.float64)
    f = np.linspace(math.sqrt(0.5) - 1, math.sqrt(2) - 1, 2001)
    f = f[np.abs(f) > 1e-3]
    want = (np.log1p(f) - f + f * f / 2) / f ** 3
    got = sum(ck * f ** k for k, ck in enumerate(c))
    assert np.abs(got - want).max() < 3e-6          # times |f|^3 <= 0.071: below 2e-7 in ln m
    assert abs(c[0] - 1.0 / 3.0) < 1e-7


def test_ln_against_libm():
    rng = np.random.default_rng(1)
    ks = np.concatenate([rng.integers(1, 2**24 + 1, size=20000),
                         [1, 2, 3, 2**24, 2**24 - 1, 2**23, 2**23 + 1, 11863283, 11863284]])
    worst = 0.0
    for k in ks:
        u = float(k) / 2.0**24
        got = oracle.ln_f32(u)
        want = math.log(u)
        worst = max(worst, abs(got - want) / max(abs(want), 1e-6))
    assert worst < 2e-7, worst
    assert oracle.ln_f32(1.0) == 0.0
    # relative accuracy right below 1, where sqrt(-2 ln u) must stay real
    for k in range(2**24 - 64, 2**24):
        u = k / 2.0**24
        assert oracle.ln_f32(u) < 0.0
        assert abs(oracle.ln_f32(u) / math.log(u) - 1.0) < 2e-7


def test_cossin_against_libm():
    rng = np.random.default_rng(2)
    ks = np.concatenate([rng.integers(0, 2**24, size=20000),
                         [0, 1, 2**22, 2**22 - 1, 2**22 + 1, 2**21, 3 * 2**21, 2**23, 3 * 2**22,
                          2**24 - 1, 5 * 2**21, 7 * 2**21]])
    worst = 0.0
    for k in ks:
        v = float(k) / 2.0**24
        c, s = oracle.cossin_2pi_f32(v)
        worst = max(worst, abs(c - math.cos(2 * math.pi * v)), abs(s - math.sin(2 * math.pi * v)))
    assert worst < 2.5e-7, worst
    assert oracle.cossin_2pi_f32(0.0) == (1.0, 0.0)
    assert oracle.cossin_2pi_f32(0.25) == (-0.0, 1.0) or oracle.cossin_2pi_f32(0.25) == (0.0, 1.0)
    assert oracle.cossin_2pi_f32(0.5)[0] == -1.0
    assert oracle.cossin_2pi_f32(0.75)[1] == -1.0


def test_normal4_is_box_muller_in_fp64_within_2e6():
    rng = np.random.default_rng(3)
    worst = 0.0
    for _ in range(20000):
        r = rng.integers(0, 2**32, size=4, dtype=np.uint64).astype(np.uint32)
        z = oracle.normal4(r)
        for h in range(2):
            u = ((int(r[2 * h]) >> 8) + 1) / 2.0**24
            v = (int(r[2 * h + 1]) >> 8) / 2.0**24
            rad = math.sqrt(-2.0 * math.log(u))
            worst = max(worst, abs(z[2 * h] - rad * math.cos(2 * math.pi * v)),
                        abs(z[2 * h + 1] - rad * math.sin(2 * math.pi * v)))
    assert worst < 2e-6, worst


def test_normal4_extremes():
    # u = 1 gives radius 0; u = 2^-24 gives the largest radius sqrt(48 ln 2)
    z = oracle.normal4([0xFFFFFFFF, 0, 0, 0])
    assert z[0] == 0.0 and z[1] == 0.0
    assert abs(float(z[2]) - math.sqrt(48 * math.log(2))) < 2e-6 and z[3] == 0.0


def test_eps_row_moments_and_layout():
    D = 200001
    eps = oracle.eps_row(12345, 3, 17, D)
    assert np.isfinite(eps).all()
    assert abs(eps.mean()) < 4.0 / math.sqrt(D)
    assert abs(eps.var() - 1.0) < 0.02
    kurt = ((eps - eps.mean()) ** 4).mean() / eps.var() ** 2
    assert abs(kurt - 3.0) < 0.1
    assert np.abs(eps).max() <= 5.77
    # layout: dims 4q..4q+3 come from counter (q, pair, generation, stream 0)
    q = 777
    z = oracle.normal4(oracle.stream_words(12345, 0, 3, 17, q))
    assert (eps[4 * q:4 * q + 4] == z).all()
    # a ragged tail drops the unused outputs
    short = oracle.eps_row(12345, 3, 17, 4 * q + 2)
    assert (short == eps[:4 * q + 2]).all()
    # different pair, generation or seed give different rows
    assert not (oracle.eps_row(12345, 3, 18, 64) == eps[:64]).any()
    assert not (oracle.eps_row(12345, 4, 17, 64) == eps[:64]).any()
    assert not (oracle.eps_row(12346, 3, 17, 64) == eps[:64]).any()
