"""Pins of the oracle's logarithm Softmax candidate (SM_LOG2: probabilities rounded to powers of two, kept as 4-bit
codes, and the shift-accumulate P V that goes with it).  The paper names the candidate (Sec. 3.2) without defining
it, so the pins are the mathematics: an independent exact-integer statement of the rounding rule, the float
Softmax it approximates, and brute force of the shift-accumulate product.  CPU only."""
import math
from fractions import Fraction

import numpy as np
import pytest

from paper_2511_15369_b200 import synth


def _codes_by_definition(orc, s, c):
    """Codes from exact integers only: e by the oracle's exponential, r = round-half-up(sum / e),
    code = the smallest k with r < 1.5 * 2^k (log2 r rounded at the arithmetic midpoint between powers of two)."""
    mx = int(s.max())
    e = [orc.softmax_exp(min(mx - int(v), c.dcap), c) for v in s]
    tot = sum(e)
    out = []
    for ej in e:
        if ej == 0:
            out.append(orc.LOG2_ZERO)
            continue
        r = math.floor(Fraction(tot, ej) + Fraction(1, 2))
        k = 0
        while not (2 * r < 3 * (1 << k)):
            k += 1
        out.append(k if k <= 15 else orc.LOG2_ZERO)
    return np.array(out, dtype=np.uint8)


@pytest.mark.parametrize("scale", [synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT, 1.0 / 700])
@pytest.mark.parametrize("n", [1, 2, 49, 197])
def test_log2_codes_match_the_exact_rule(orc, scale, n):
    c = orc.softmax_prepare(scale, n, 4, orc.SM_LOG2)
    s = synth.quantize_scores(synth.softmax_logits(24, n, seed=n), scale)
    got = orc.softmax(s, c)
    for i in range(s.shape[0]):
        assert (got[i] == _codes_by_definition(orc, s[i], c)).all()
    assert ((got <= 15) | (got == orc.LOG2_ZERO)).all()
    assert (got[np.arange(s.shape[0]), s.argmax(axis=1)] <= 8).all()        # the row maximum is never dropped


def test_log2_tracks_the_float_softmax(orc):
    n, S = 197, synth.SOFTMAX_SCALE_ACC
    s = synth.quantize_scores(synth.softmax_logits(64, n, seed=2), S)
    codes = orc.softmax(s, orc.softmax_prepare(S, n, 4, orc.SM_LOG2)).astype(np.int64)
    z = s * S
    p = np.exp(z - z.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    live = codes != orc.LOG2_ZERO
    big = p >= 2.0 ** -12
    assert live[big].all()                                                   # representable probabilities are kept
    # the rule rounds up from 1.5 * 2^k on, so the code is off by at most log2(1.5) = 0.585 octaves; the polynomial
    # exponential and the integer rounding of sum / e add a little
    assert np.abs(-codes[big] - np.log2(p[big])).max() <= math.log2(1.5) + 0.03
    assert (p[~live] < 2.0 ** -14.4).all()                                   # what is dropped is below 2^-15 * 1.5
    tot = np.where(live, 2.0 ** -codes.astype(np.float64), 0.0).sum(axis=1)
    assert (tot > 0.70).all() and (tot < 1.42).all()                         # sum of the powers of two: within sqrt 2
    # a single-entry row is probability one: code 0
    assert orc.softmax(np.array([[7]], dtype=np.int32), orc.softmax_prepare(S, 1, 4, orc.SM_LOG2))[0, 0] == 0
    # two equal entries: 1/2 each
    assert orc.softmax(np.array([[5, 5]], dtype=np.int32), orc.softmax_prepare(S, 2, 4, orc.SM_LOG2)).tolist() == [[1, 1]]
    with pytest.raises(orc.OracleError):
        orc.softmax_prepare(S, n, 8, orc.SM_LOG2)                            # codes are 4 bits wide


def test_log2_attention_is_shift_accumulate(orc):
    rng = np.random.default_rng(4)
    B, H, N, dh = 2, 3, 21, 16
    q = rng.integers(-128, 128, size=(B, H, N, dh)).astype(np.int8)
    k = rng.integers(-128, 128, size=(B, H, N, dh)).astype(np.int8)
    v = rng.integers(-128, 128, size=(B, H, N, dh)).astype(np.int8)
    sc = orc.softmax_prepare(2.0e-4, N, 4, orc.SM_LOG2)
    rq = orc.requant_prepare(2.0 ** -15 * 0.9)
    got = orc.attention_block(q, k, v, sc, rq)
    for b in range(B):
        for h in range(H):
            s = q[b, h].astype(np.int64) @ k[b, h].astype(np.int64).T
            codes = orc.softmax(s.astype(np.int32), sc)
            for i in range(N):
                for d in range(dh):
                    acc = sum(int(v[b, h, j, d]) << (15 - int(codes[i, j])) for j in range(N) if codes[i, j] != orc.LOG2_ZERO)
                    assert got[b, i, h * dh + d] == orc.requant(acc, rq)
