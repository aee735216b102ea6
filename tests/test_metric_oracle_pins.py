"""Pins of the Unified-Metric oracle (Sec. 3.5, Eqs. (16)-(20)): the worked SQNR example the paper prints, closed
forms of the Softplus and of the harmonic-mean term, the textbook noise power of a uniform quantiser, brute force
with exact rationals, and the identities of the float layers.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import metric

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def test_sqnr_worked_example():
    g = _golden("sqnr_example.txt")
    assert metric.sqnr_db(g["signal_power"], g["noise_a"]) == pytest.approx(g["sqnr_a_db"], abs=1e-12)
    b = metric.sqnr_db(g["signal_power"], g["noise_b"])
    assert 0.0 <= b - g["sqnr_b_db"] < 0.01                    # printed with two decimals, cut off
    # the "20 log" the equation prints would give 40 dB and 44.4 dB: excluded by the example
    assert abs(20.0 * math.log10(g["signal_power"] / g["noise_a"]) - g["sqnr_a_db"]) > 10.0
    # a ratio of means equals the ratio of sums
    x = np.array([3.0, -4.0, 12.0]); q = np.array([2.0, -4.5, 12.25])
    sx2, se2 = metric.error_sums(x, q)
    assert metric.sqnr_db(sx2, se2) == pytest.approx(10 * math.log10(np.mean(x * x) / np.mean((x - q) ** 2)), abs=1e-12)


def test_softplus_closed_forms():
    assert metric.softplus(0.0) == pytest.approx(math.log(2.0), abs=1e-15)
    for v in (-30.0, -3.0, -0.1, 0.2, 5.0, 40.0, 800.0):
        assert metric.softplus(v) - metric.softplus(-v) == pytest.approx(v, rel=1e-12, abs=1e-12)   # N(v) - N(-v) = v
        assert metric.softplus(v) >= max(v, 0.0)
    assert metric.softplus(1.0) == pytest.approx(math.log(1.0 + math.e), abs=1e-15)
    assert metric.softplus(800.0) == 800.0 and math.isfinite(metric.softplus(1e308))
    assert metric.softplus(-800.0) == pytest.approx(0.0, abs=1e-300)
    vs = np.linspace(-20, 20, 401)
    ns = [metric.softplus(v) for v in vs]
    assert all(b > a for a, b in zip(ns, ns[1:]))


def test_layer_term_harmonic_mean():
    # equal factors a = 1/N(Q) = N(P) = N(C): the term is 1/a
    a = math.log(2.0)                                  # N(0)
    q = math.log(math.expm1(1.0 / a))                  # N(q) = 1/a
    assert metric.softplus(q) == pytest.approx(1.0 / a, rel=1e-14)
    assert metric.layer_term(q, 0.0, 0.0) == pytest.approx(1.0 / a, rel=1e-14)
    # harmonic mean of (N(Q), 1/N(P), 1/N(C)) written out
    Q, P, Cops, unit = 31.5, 0.37, 2.4e6, 1.0e6
    f = [metric.softplus(Q), 1.0 / metric.softplus(P), 1.0 / metric.softplus(Cops / unit)]
    assert metric.layer_term(Q, P, Cops, unit) == pytest.approx(3.0 / sum(1.0 / v for v in f), rel=1e-14)
    # better sensitivity, smaller perturbation, smaller cost: each raises the term
    base = metric.layer_term(Q, P, Cops, unit)
    assert metric.layer_term(Q + 3, P, Cops, unit) > base
    assert metric.layer_term(Q, P / 2, Cops, unit) > base
    assert metric.layer_term(Q, P, Cops / 2, unit) > base
    # an exact candidate (no error at all) has a finite term
    assert math.isfinite(metric.layer_term(math.inf, 0.0, Cops, unit))
    assert metric.unified_metric([0.25, 0.5, 1.0]) == 1.75


def test_error_sums_exact_rationals():
    rng = np.random.default_rng(0)
    x = rng.integers(-1000, 1000, size=50) / 64.0
    q = rng.integers(-1000, 1000, size=50) / 128.0
    sx2 = sum(Fraction(float(v)) ** 2 for v in x)
    se2 = sum((Fraction(float(a)) - Fraction(float(b))) ** 2 for a, b in zip(x, q))
    got = metric.error_sums(x, q)
    assert got[0] == float(sx2) and got[1] == float(se2)
    assert metric.error_sums(x, x) == (float(sx2), 0.0)
    assert metric.sqnr_db(*metric.error_sums(x, x)) == math.inf
    # asymmetric in (X, Q): the signal power is that of the first argument
    assert metric.error_sums(q, x)[0] != got[0] and metric.error_sums(q, x)[1] == got[1]


def test_uniform_quantiser_noise_power():
    # X uniform on [-1, 1), rounded to a grid of step d: noise power d^2/12, signal power 1/3 (textbook)
    rng = np.random.default_rng(1)
    x = rng.uniform(-1.0, 1.0, size=1 << 20)
    for bits in (4, 6, 8):
        d = 2.0 / (1 << bits)
        q = np.round(x / d) * d
        want = 10.0 * math.log10((1.0 / 3.0) / (d * d / 12.0))       # = 6.02 bits dB
        assert want == pytest.approx(6.0206 * bits, abs=1e-3)
        got_q, got_p, _ = metric.evaluate(x, q, 1.0)
        assert got_q == pytest.approx(want, abs=0.05)
        assert got_p == pytest.approx(x.size * d * d / 12.0, rel=0.01)


def test_float_layers_identities():
    rng = np.random.default_rng(2)
    s = rng.integers(-40000, 40000, size=(7, 33))
    p = metric.softmax_float(s, 3e-4)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-14) and (p > 0).all()
    assert np.allclose(metric.softmax_float(s + 12345, 3e-4), p, atol=1e-15)          # shift invariance
    r = p[:, :1] / p[:, 1:2]
    assert np.allclose(np.log(r), (s[:, :1] - s[:, 1:2]) * 3e-4, atol=1e-12)           # ratios are exp of differences
    x = rng.integers(-30000, 30000, size=1000)
    S = 1.3e-4
    g = metric.gelu_float(x, S)
    assert np.allclose(g - metric.gelu_float(-x, S), x * S, atol=1e-14)                 # GELU(v) - GELU(-v) = v
    assert metric.gelu_float(np.array([0]), S)[0] == 0.0
    assert metric.gelu_float(np.array([1]), 1.0)[0] == pytest.approx(0.5 * (1 + math.erf(1 / math.sqrt(2))), abs=1e-15)
    assert metric.gelu_float(np.array([40000]), 1e-3)[0] == pytest.approx(40.0, abs=1e-12)
    xl = rng.integers(-128, 128, size=(5, 96))
    one, zero = np.ones(96), np.zeros(96)
    y = metric.layernorm_float(xl, one, zero)
    assert np.allclose(y.mean(axis=1), 0.0, atol=1e-13) and np.allclose((y * y).mean(axis=1), 1.0, atol=1e-12)
    gam, bet = rng.normal(1, 0.1, 96), rng.normal(0, 0.1, 96)
    assert np.allclose(metric.layernorm_float(xl, gam, bet), y * gam + bet, atol=1e-13)
    assert np.allclose(metric.layernorm_float(3 * xl + 7, gam, bet), metric.layernorm_float(xl, gam, bet), atol=1e-12)
    const = np.full((2, 96), 5)
    assert np.array_equal(metric.layernorm_float(const, gam, bet), np.broadcast_to(bet, (2, 96)))
    sh = rng.integers(0, 4, size=96)
    assert np.allclose(metric.layernorm_float(xl, gam, bet, sh), metric.layernorm_float(xl * (1 << sh), gam, bet), atol=1e-12)


def test_dequantisers_and_counts():
    assert metric.softmax_deq(np.array([0, 64, 128]), 8).tolist() == [0.0, 0.5, 1.0]
    assert metric.softmax_deq(np.array([8]), 4).tolist() == [1.0]
    assert metric.affine_deq(np.array([-128, -100, 27]), 0.03, -100).tolist() == [-28 * 0.03, 0.0, 127 * 0.03]
    # counts grow linearly with the tensor and order the candidates as their definitions do
    for kind in (metric.SOFTMAX, metric.GELU, metric.LAYERNORM):
        for v in (0, 1, 2):
            assert metric.op_count(kind, v, 20, 64) == 2 * metric.op_count(kind, v, 10, 64)
    sm = [metric.op_count(metric.SOFTMAX, v, 197, 197) for v in (0, 1, 2)]
    assert sm[0] > sm[1] > sm[2]                              # Bit-exp adds three shift-add terms to Shiftmax
    ge = [metric.op_count(metric.GELU, v, 197, 768) for v in (0, 1, 2)]
    assert ge[2] > ge[0] > ge[1]
    assert metric.select([0.1, 0.7, 0.7, 0.2]) == 1 and metric.select([0.3]) == 0


def test_integer_candidates_through_the_metric():
    """The three Softmax candidates on the paper-like logits: all are usable approximations (SQNR well above 10 dB)
    and the metric ranks them without error."""
    import oracle
    from paper_2511_15369_b200 import synth
    n = 197
    s = synth.quantize_scores(synth.softmax_logits(64, n, seed=0), synth.SOFTMAX_SCALE_ACC)
    x = metric.softmax_float(s, synth.SOFTMAX_SCALE_ACC)
    terms = []
    for v in (0, 1, 2):
        c = oracle.softmax_prepare(synth.SOFTMAX_SCALE_ACC, n, 8, v)
        q, p, t = metric.evaluate(x, metric.softmax_deq(oracle.softmax(s, c), 8), metric.op_count(metric.SOFTMAX, v, 64, n))
        assert q > 15.0 and 0.0 < t < 3.0 / math.log(2.0)
        terms.append(t)
    assert 0 <= metric.select(terms) < 3
