"""Pins of the CPU oracle against what the paper and the mathematics fix.

Every test here runs on the CPU.  The checks are chosen so that a plausible
mistake in the oracle (a dropped term, a wrong sign, a wrong shift, a
transposed operand) fails at least one of them:
  * values the paper prints (Table 3: erf / GELU approximation errors on (-3, 3);
    Table 5: base-2 exponential errors on (-1, 1); the coefficients of Eq. (3));
  * exact big-integer transcriptions evaluated by brute force;
  * invariants of Eq. (15) (row-sum bound, monotone IntDiv) and of Eq. (9);
  * special cases that reduce to textbook routines (math.isqrt, fp64 LayerNorm,
    int64 matmul).
"""
import math
import os

import numpy as np
import pytest

from paper_2511_15369_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    """golden/*.txt: lines of 'key value  # citation'."""
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


# ------------------------------------------------------------------ R (dyadic requant)

def _py_requant(y, mult, shift, zp, lo, hi):
    v = (((y * mult) >> 32) + (1 << (shift - 1))) >> shift   # Python ints: >> is floor
    return max(lo, min(hi, v + zp))


def test_requant_matches_bigint_and_ideal(orc):
    rng = np.random.default_rng(1)
    worst = 0.0
    for _ in range(300):
        ratio = float(2.0 ** rng.uniform(-30, -2.01))
        rq = orc.requant_prepare(ratio, zp=int(rng.integers(-5, 6)), qmin=-(1 << 30), qmax=1 << 30)
        assert (1 << 30) <= rq.mult < (1 << 31) and 1 <= rq.shift <= 31
        assert abs(rq.mult * 2.0 ** -(32 + rq.shift) / ratio - 1) < 2 ** -29
        ys = list(rng.integers(-(1 << 31), 1 << 31, size=40)) + [0, 1, -1, (1 << 31) - 1, -(1 << 31)]
        for y in ys:
            y = int(y)
            got = orc.requant(y, rq)
            assert got == _py_requant(y, rq.mult, rq.shift, rq.zp, rq.qmin, rq.qmax)
            worst = max(worst, abs(got - rq.zp - math.floor(y * ratio + 0.5)))
    assert worst <= 1          # floor-then-round differs from round-to-nearest by at most 1


def test_requant_clamps_and_rejects(orc):
    rq = orc.requant_prepare(0.1, zp=3, qmin=-128, qmax=127)
    assert orc.requant(10 ** 9, rq) == 127 and orc.requant(-10 ** 9, rq) == -128
    assert orc.requant(0, rq) == 3
    for bad in (0.25, 0.3, 0.0, -1.0, 2.0 ** -34):
        with pytest.raises(orc.OracleError):
            orc.requant_prepare(bad)


# ------------------------------------------------------------------ Softmax: the exponential

def test_table5_base2_exp_errors():
    """Table 5: L2 (RMS) / Linf error of the two first-degree forms of 2^x on (-1, 1)."""
    g = _golden("table5_exp2_error.txt")
    x = np.linspace(-1, 1, 600001)[1:-1]
    t = 2.0 ** x
    ivit = 1 + x / 2
    ours = 1 + math.log(2) * x
    assert abs(np.sqrt(np.mean((t - ivit) ** 2)) - g["ivit_l2"]) < 1e-4
    assert abs(np.abs(t - ivit).max() - g["ivit_linf"]) < 1e-4
    assert abs(np.sqrt(np.mean((t - ours) ** 2)) - g["ours_l2"]) < 1e-4
    assert abs(np.abs(t - ours).max() - g["ours_linf"]) < 1e-4


def _py_exp(d, x0, nsh, variant):
    """Big-int transcription of Eqs. (7)-(10), (13)-(14); Python's >> floors."""
    Qd = -d
    Qp = Qd + (Qd >> 1) - (Qd >> 4)
    P = -Qp
    q, r = divmod(P, x0)
    u = -r
    base = ((u >> 1) + (u >> 3) + (u >> 4) + x0) if variant == 0 else ((u >> 1) + x0)
    return 0 if q > 31 else ((base << nsh) >> q)


@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("scale", [1 / 10.5, 1 / 50.5, 1 / 255.5, 3e-4])
def test_exp_core_bruteforce(orc, variant, scale):
    c = orc.softmax_prepare(scale, 197, 8, variant)
    x0 = c.x0
    assert x0 == math.floor(1 / scale) and c.dcap == 34 * x0
    assert (1 << 13) <= (x0 << c.nsh) < (1 << 14)
    prev = None
    for d in range(0, c.dcap + 1):
        e = orc.softmax_exp(d, c)
        assert e == _py_exp(d, x0, c.nsh, variant)
        assert e >= 0
        if prev is not None and variant == 1:
            assert e <= prev       # 1 + x/2 is continuous across octaves: globally monotone
        prev = e
    assert orc.softmax_exp(0, c) == x0 << c.nsh          # e(0) is the integer 1.0
    assert orc.softmax_exp(c.dcap, c) == 0               # beyond the cap the value is 0 anyway


def test_exp_core_large_x0_sampled(orc):
    c = orc.softmax_prepare(1.0 / ((1 << 20) - 2.5), 49, 8, 0)
    assert c.x0 == (1 << 20) - 3 and c.nsh == 0
    rng = np.random.default_rng(3)
    for d in [0, 1, c.dcap, c.dcap - 1] + [int(v) for v in rng.integers(0, c.dcap, size=20000)]:
        assert orc.softmax_exp(d, c) == _py_exp(d, c.x0, 0, 0)


def test_exp_against_true_exponential(orc):
    """The integer form against exp(-S d): error budget = first-degree fraction
    (|2^x - (1 + 0.6875 x)| <= 0.1875 on (-1, 0]) + the 1.4375 ~ log2(e) constant."""
    S = 3e-4
    for variant, lo, hi in ((0, 0.17, 0.23), (1, 0.03, 0.06)):
        c = orc.softmax_prepare(S, 197, 8, variant)
        unit = c.x0 << c.nsh
        d = np.arange(0, 12 * c.x0)
        e = np.array([orc.softmax_exp(int(v), c) for v in d]) / unit
        err = np.abs(e - np.exp(-S * d)).max()
        assert lo < err < hi, err
        # at an octave boundary the value is exactly 2^-q: pins the 1 + 1/2 - 1/16 constant of Eq. (7)
        for q in (1, 2, 5):
            dq = math.ceil(q * c.x0 / 1.4375)
            assert abs(orc.softmax_exp(dq, c) / unit * 2 ** q - 1) < 0.01
            assert abs(math.exp(-S * dq) * 2 ** q - 1) < 0.01 * q


def test_bitexp_monotone_inside_octaves_only(orc):
    """Eq. (13) drops to 0.3125 at the end of an octave while the next one starts at 0.5:
    one upward jump per octave, of ratio <= 0.5 / 0.3125; monotone elsewhere."""
    c = orc.softmax_prepare(3e-4, 197, 8, 0)
    e = [orc.softmax_exp(d, c) for d in range(0, 16 * c.x0)]
    ups = [(i, e[i - 1], e[i]) for i in range(1, len(e)) if e[i] > e[i - 1]]
    assert 8 <= len(ups) <= 24
    for _, a, b in ups:
        assert b <= 0.5 / 0.3125 * a + 4        # + integer rounding of both sides
    assert ups[0][0] == 2319 and (ups[0][1], ups[0][2]) == (1041 * 4, 1665 * 4)


# ------------------------------------------------------------------ Softmax: rows

@pytest.mark.parametrize("variant,tol", [(0, 0.085), (1, 0.03), (2, 0.02)])
@pytest.mark.parametrize("scale", [synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT])
@pytest.mark.parametrize("n", [49, 197])
def test_softmax_rows_invariants_and_accuracy(orc, variant, tol, scale, n):
    logits = synth.softmax_logits(64, n, seed=5)
    s = synth.quantize_scores(logits, scale)
    c = orc.softmax_prepare(scale, n, 8, variant)
    p = orc.softmax(s, c)
    sums = p.astype(np.int64).sum(axis=1)
    assert (sums <= 128).all()                      # each term is a floor of a share of 2^(b-1)
    assert (sums > 128 - n - 1).all()
    ref = synth.softmax_ref(s * scale)
    assert np.abs(p / 128.0 - ref).max() < tol
    # the arg-max of a row keeps the largest probability
    assert (p[np.arange(64), s.argmax(axis=1)] == p.max(axis=1)).all()


def test_softmax_small_cases(orc):
    c = orc.softmax_prepare(3e-4, 1, 8, 0)
    assert orc.softmax(np.array([[123456]], dtype=np.int32), c)[0, 0] in (127, 128)
    c = orc.softmax_prepare(3e-4, 4, 8, 0)
    p = orc.softmax(np.array([[7, 7, 7, 7]], dtype=np.int32), c)
    assert (p == 32).all() or (p == 31).all()
    # one huge outlier takes everything
    p = orc.softmax(np.array([[0, (1 << 30) - 1, -(1 << 30) + 1, 5]], dtype=np.int32), c)
    assert p[0, 1] in (127, 128) and p[0, 0] == 0 and p[0, 2] == 0
    # out_bits: scale of the output is 2^-(b-1)
    for b in (4, 6, 8):
        cb = orc.softmax_prepare(3e-4, 4, b, 0)
        p = orc.softmax(np.array([[0, 0, 0, 0]], dtype=np.int32), cb)
        assert p.max() <= 1 << (b - 1) and abs(int(p.sum()) - (1 << (b - 1))) <= 4


def test_softmax_bias_and_mask(orc):
    rng = np.random.default_rng(9)
    c = orc.softmax_prepare(3e-4, 49, 8, 0)
    s = rng.integers(-20000, 20000, size=(12, 49)).astype(np.int32)
    bias = rng.integers(-5000, 5000, size=(3, 49)).astype(np.int32)
    got = orc.softmax(s, c, bias=bias, bias_period=3)
    want = orc.softmax((s + bias[np.arange(12) % 3]).astype(np.int32), c)
    assert (got == want).all()
    # masked entries: probability 0, excluded from the maximum and from the sum
    row = s[0].astype(np.int64)
    mask = np.zeros(49, dtype=np.uint8)
    mask[::3] = 1
    pm = orc.softmax_row(row, c, mask)
    assert (pm[mask == 1] == 0).all()
    keep = np.flatnonzero(mask == 0)
    c_small = orc.softmax_prepare(3e-4, 49, 8, 0)
    sub = orc.softmax_row(row[keep], c_small)
    assert (pm[keep] == sub).all()


def test_softmax_poly_variant(orc):
    """The polynomial candidate: a(p+b)^2+c of the cited work reproduces exp on (-ln2, 0]."""
    a, b, cc = 0.3585, 1.353, 0.344
    p = np.linspace(-math.log(2), 0, 20001)
    assert np.abs(a * (p + b) ** 2 + cc - np.exp(p)).max() < 3e-3
    S = 3e-4
    c = orc.softmax_prepare(S, 197, 8, 2)
    assert c.qln2 == math.floor(math.log(2) / S) and c.qb == math.floor(b / S)
    unit = orc.softmax_exp(0, c)
    assert (1 << 13) <= unit < (1 << 14)
    d = np.arange(0, 10 * c.x0, 7)
    e = np.array([orc.softmax_exp(int(v), c) for v in d]) / unit
    assert np.abs(e - np.exp(-S * d)).max() < 6e-3


def test_softmax_prepare_constants(orc):
    g = _golden("softmax_consts.txt")
    c = orc.softmax_prepare(3e-4, 197, 8, 0)
    assert (c.x0, c.nsh, c.M) == (g["x0_acc"], g["N_acc"], g["M_acc_197"])
    assert orc.softmax_prepare(3e-4, 49, 8, 0).M == g["M_acc_49"]
    c = orc.softmax_prepare(12 / 127, 197, 8, 0)
    assert (c.x0, c.nsh, c.M) == (g["x0_8bit"], g["N_8bit"], g["M_8bit_197"])
    for bad in (0.2, 1e-9):
        with pytest.raises(orc.OracleError):
            orc.softmax_prepare(bad, 197, 8, 0)


# ------------------------------------------------------------------ GELU

def _gelu_sweep(orc, variant, S, in_bits):
    c = orc.gelu_prepare(S, in_bits, 0.05, 0, 8, variant)
    lo, hi = -(1 << (in_bits - 1)), (1 << (in_bits - 1)) - 1
    xs = np.arange(lo, hi + 1)
    core = np.array([orc.gelu_core(int(v), c) for v in xs], dtype=np.float64)
    return c, xs, core, orc.gelu_core_scale(S, c)


@pytest.mark.parametrize("variant,key", [(0, "ours"), (1, "ibert")])
def test_table3_erf_and_gelu_errors_from_the_integer_pipeline(orc, variant, key):
    """Table 3 on (-3, 3), reproduced from the oracle's integer GELU at a fine 16-bit scale:
    GELU error directly; erf error from L = 2*GELU/x - 1 evaluated at x / sqrt(2)."""
    g = _golden("table3_erf_gelu_error.txt")
    S = 8.6 / 65535          # covers x / sqrt(2) in (-3, 3); floor(|b| / S') stays below 2^15
    c, xs, core, Sy = _gelu_sweep(orc, variant, S, 16)
    x = xs * S
    inside = np.abs(x) < 3
    approx = core * Sy
    err = approx[inside] - synth.gelu_ref(x[inside])
    assert abs(np.abs(err).max() - g[key + "_gelu_linf"]) < 3e-4
    assert abs(np.sqrt(np.mean(err ** 2)) - g[key + "_gelu_l2"]) < 2e-4
    # erf: u = x / sqrt(2) in (-3, 3)
    u = x / math.sqrt(2)
    sel = (np.abs(u) < 3) & (xs != 0)
    L = 2 * approx[sel] / x[sel] - 1
    erf = np.vectorize(math.erf)(u[sel])
    e2 = L - erf
    assert abs(np.abs(e2).max() - g[key + "_erf_linf"]) < 1.5e-3
    assert abs(np.sqrt(np.mean(e2 ** 2)) - g[key + "_erf_l2"]) < 3e-4


def test_gelu_quartic_constants(orc):
    """Eq. (3): a = -0.019913, b = -2.698088; a*b^4 + 1 is the erf error at 0 (Table 3's Linf)."""
    g = _golden("table3_erf_gelu_error.txt")
    a, b = -0.019913, -2.698088
    assert abs(abs(a * b ** 4 + 1) - g["ours_erf_linf"]) < 5e-4
    S = 1e-3
    c = orc.gelu_prepare(S, 16, 0.05, 0, 8, 0)
    Sp = S / math.sqrt(2)
    assert c.Bq == math.floor(-b / Sp)
    assert abs(c.C * 4.0 ** c.sh2 * (-a) * Sp ** 4 - 1) < 1e-6


@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("in_bits,S", [(8, 8.0 / 127), (8, 3.0 / 127), (12, 0.003), (16, 1.2e-4)])
def test_gelu_exhaustive_properties(orc, variant, in_bits, S):
    c, xs, core, Sy = _gelu_sweep(orc, variant, S, in_bits)
    assert np.abs(core).max() < 2 ** 31
    G1 = (2 * c.C) >> c.gs
    for x, y in zip(xs, core):
        if x >= c.Bq:
            assert y == x * G1            # saturated: GELU(x) = x
        if x <= -c.Bq:
            assert y == 0                 # saturated: GELU(x) = 0
    # accuracy against fp64 GELU over the whole input range (coarser scales lose a little)
    bound = {0: 0.0135, 1: 0.0215}[variant]
    assert np.abs(core * Sy - synth.gelu_ref(xs * S)).max() < bound
    # G(x) + G(-x) = 2C: y(x)/x + y(-x)/(-x) is constant where the shift loses nothing
    if c.gs == 0:
        for x in (1, 5, c.Bq // 2):
            assert orc.gelu_core(x, c) // x + orc.gelu_core(-x, c) // -x == 2 * c.C


def test_gelu_out_of_range_input_is_clamped(orc):
    c = orc.gelu_prepare(0.01, 12, 0.05, 0, 8, 0)
    assert orc.gelu_core(10 ** 6, c) == orc.gelu_core(2047, c)
    assert orc.gelu_core(-10 ** 6, c) == orc.gelu_core(-2048, c)


def test_gelu_shift_variant(orc):
    """x * sigmoid(1.702 x) with the shift exponential: within the exp error of the sigmoid form."""
    S = 2e-3
    c, xs, core, Sy = _gelu_sweep(orc, 2, S, 12)
    x = xs * S
    target = x / (1 + np.exp(-1.6875 * x))
    assert np.abs(core * Sy - target).max() < 0.02
    assert np.abs(core * Sy - synth.gelu_ref(x)).max() < 0.04


def test_gelu_requantised_output(orc):
    x = synth.gelu_values(20000, seed=2)
    xq, S = synth.quantize_sym(x, 16)
    ref = synth.gelu_ref(xq * S)
    So, zp = synth.affine_out_quant(ref)
    for variant, tol in ((0, 1.0), (1, 1.6), (2, 2.5)):
        Sv, xv = (S, xq) if variant != 2 else synth.quantize_sym(x, 12)[::-1]
        c = orc.gelu_prepare(Sv, 16 if variant != 2 else 12, So, zp, 8, variant)
        y = orc.gelu(xv.astype(np.int32), c)
        refv = synth.gelu_ref(xv * Sv)
        want = np.clip(np.round(refv / So) + zp, -128, 127)
        assert np.abs(y - want).max() <= math.ceil(tol + 0.0135 / So)


# ------------------------------------------------------------------ LayerNorm

def test_isqrt_variants(orc):
    rng = np.random.default_rng(4)
    vals = list(range(0, 1 << 16)) + [int(v) for v in rng.integers(0, 1 << 41, size=100000)]
    vals += [(k * k) + j for k in (3, 1000, 46341, 1 << 20) for j in (-1, 0, 1)] + [(1 << 41), (1 << 52) - 1]
    for V in vals:
        s = math.isqrt(V)
        assert orc.isqrt(V, orc.LN_NEWTON) == s
        assert orc.isqrt(V, orc.LN_PTF) == s
        assert orc.isqrt(V, orc.LN_SHIFT) - s in (0, 1)
    # the fixed-step form really can stop one above: V + 1 a perfect square
    assert any(orc.isqrt(k * k - 1, orc.LN_SHIFT) == k for k in range(2, 2000))


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("dim", [96, 192, 768])
def test_layernorm_against_fp64(orc, variant, dim):
    xf, gamma, beta, _ = synth.ln_values(200, dim, seed=7)
    xq, S = synth.quantize_sym(xf, 8, np.int8)
    ptf = synth.ptf_shifts(xq) if variant == orc.LN_PTF else None
    xeff = xq.astype(np.float64) * (2.0 ** ptf if ptf is not None else 1.0)
    ref = synth.layernorm_ref(xeff, gamma.astype(np.float64), beta.astype(np.float64))
    So, zp = synth.affine_out_quant(ref)
    gq, bq, c = orc.layernorm_prepare(gamma, beta, So, zp, 8, variant)
    y = orc.layernorm(xq, gq, bq, c, ptf)
    want = np.clip(np.round(ref / So) + zp, -128, 127)
    assert np.abs(y - want).max() <= 1
    assert np.abs(y - want).mean() < 0.05


def test_layernorm_constant_row_and_scale_invariance(orc):
    gamma = np.linspace(0.5, 1.5, 64).astype(np.float32)
    beta = np.linspace(-0.3, 0.3, 64).astype(np.float32)
    gq, bq, c = orc.layernorm_prepare(gamma, beta, 0.02, 0, 8, orc.LN_NEWTON)
    x = np.full((1, 64), 17, dtype=np.int8)
    y = orc.layernorm(x, gq, bq, c)
    assert (y[0] == [orc.requant(int(b), c.out) for b in bq]).all()     # zero variance: output = R(beta)
    # the input scale cancels: doubling x changes nothing beyond rounding
    rng = np.random.default_rng(0)
    a = rng.integers(-60, 60, size=(8, 64)).astype(np.int8)
    y1 = orc.layernorm(a, gq, bq, c)
    y2 = orc.layernorm((2 * a).astype(np.int8), gq, bq, c)
    assert np.abs(y1.astype(int) - y2.astype(int)).max() <= 1


# ------------------------------------------------------------------ GEMM carriers and blocks

def _np_requant_vec(acc, mult, shift):
    acc = acc.astype(object)
    out = np.empty(acc.shape, dtype=object)
    for n in range(acc.shape[1]):
        m, s = int(mult[n]), int(shift[n])
        out[:, n] = [(((int(a) * m) >> 32) + (1 << (s - 1))) >> s for a in acc[:, n]]
    return out.astype(np.int64)


def _prep_channels(orc, ratios):
    rqs = [orc.requant_prepare(float(r)) for r in ratios]
    return (np.array([r.mult for r in rqs], dtype=np.int32), np.array([r.shift for r in rqs], dtype=np.int8))


@pytest.mark.parametrize("w_bits", [8, 4])
def test_linear_against_int64_matmul(orc, w_bits):
    rng = np.random.default_rng(11)
    M, N, K = 37, 24, 64
    x = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    lim = 8 if w_bits == 4 else 128
    w = rng.integers(-lim, lim, size=(N, K)).astype(np.int8)
    bias = rng.integers(-1000, 1000, size=N).astype(np.int32)
    mult, shift = _prep_channels(orc, 2.0 ** rng.uniform(-9, -5, size=N))
    res = rng.integers(-128, 128, size=(M, N)).astype(np.int8)
    rrq = orc.requant_prepare(0.7 / 65536, zp=-3)
    wp = synth.pack_int4(w) if w_bits == 4 else w
    y = orc.linear(x, wp, bias, mult, shift, out_zp=5, residual=res, residual_rq=rrq, w_bits=w_bits)
    acc = x.astype(np.int64) @ w.astype(np.int64).T + bias
    main = _np_requant_vec(acc, mult, shift)
    rr = (res.astype(np.int64) + 3) << 16
    rterm = _np_requant_vec(rr, np.full(N, rrq.mult), np.full(N, rrq.shift))
    want = np.clip(main + rterm + 5, -128, 127)
    assert (y == want).all()
    y0 = orc.linear(x, wp, None, mult, shift, w_bits=w_bits)
    assert (y0 == np.clip(_np_requant_vec(acc - bias, mult, shift), -128, 127)).all()
    # narrower activations (the W6A6 setting): the same sum, clamped to the out_bits range
    for bits in (6, 4):
        yb = orc.linear(x, wp, bias, mult, shift, out_zp=5, residual=res, residual_rq=rrq, w_bits=w_bits, out_bits=bits)
        assert (yb == np.clip(main + rterm + 5, -(1 << (bits - 1)), (1 << (bits - 1)) - 1)).all()
        assert yb.min() == -(1 << (bits - 1)) and yb.max() == (1 << (bits - 1)) - 1


def test_attention_against_composition(orc):
    rng = np.random.default_rng(12)
    B, H, N, dh = 2, 3, 21, 16
    q, k, v = (rng.integers(-128, 128, size=(B, H, N, dh)).astype(np.int8) for _ in range(3))
    bias = rng.integers(-3000, 3000, size=(H, N, N)).astype(np.int32)
    mask_id = rng.integers(0, 2, size=(B, N)).astype(np.uint8)
    sc = orc.softmax_prepare(4e-4, N, 8, 0)
    rq = orc.requant_prepare(0.01, zp=2)
    for use_bias, use_mask in ((0, 0), (1, 0), (1, 1)):
        out = orc.attention_block(q, k, v, sc, rq, bias if use_bias else None, mask_id if use_mask else None)
        for b in range(B):
            for h in range(H):
                S = q[b, h].astype(np.int64) @ k[b, h].astype(np.int64).T + (bias[h] if use_bias else 0)
                for i in range(N):
                    m = (mask_id[b] != mask_id[b, i]).astype(np.uint8) if use_mask else None
                    p = orc.softmax_row(S[i], sc, m).astype(np.int64)
                    o = p @ v[b, h].astype(np.int64)
                    want = [orc.requant(int(t), rq) for t in o]
                    assert (out[b, i, h * dh:(h + 1) * dh] == want).all()


def _prepared_block(orc, spec):
    sh = spec.shape

    def lin(ls):
        m, s = _prep_channels(orc, ls.ratio)
        return m, s

    d = dict(B=sh.B, N=sh.N, D=sh.D, H=sh.H, dh=sh.dh, Dh=sh.Dh, w_bits=spec.w_bits)
    g1, b1, c1 = orc.layernorm_prepare(spec.ln1["gamma"], spec.ln1["beta"], spec.ln1["out_scale"], spec.ln1["out_zp"])
    g2, b2, c2 = orc.layernorm_prepare(spec.ln2["gamma"], spec.ln2["beta"], spec.ln2["out_scale"], spec.ln2["out_zp"])
    d.update(ln1_gamma=g1, ln1_beta=b1, ln1=c1, ln2_gamma=g2, ln2_beta=b2, ln2=c2)
    for name, ls in (("qkv", spec.qkv), ("proj", spec.proj), ("fc1", spec.fc1), ("fc2", spec.fc2)):
        m, s = lin(ls)
        d["w_" + name], d["b_" + name], d["m_" + name], d["s_" + name] = ls.w_packed, ls.bias, m, s
    d["sm"] = orc.softmax_prepare(spec.softmax_scale, sh.N, 8, 0)
    d["pv_rq"] = orc.requant_prepare(spec.pv_ratio)
    d["attn_bias"], d["mask_id"] = spec.attn_bias, spec.mask_id
    d["res1_rq"] = orc.requant_prepare(spec.proj.res_ratio / 65536, zp=spec.proj.res_zp)
    d["res2_rq"] = orc.requant_prepare(spec.fc2.res_ratio / 65536, zp=spec.fc2.res_zp)
    gl = spec.gelu
    d["gelu"] = orc.gelu_prepare(gl["in_scale"], gl["in_bits"], gl["out_scale"], gl["out_zp"], 8, 0)
    d["proj_zp"], d["fc2_zp"] = spec.proj.out_zp, spec.fc2.out_zp
    return d


@pytest.mark.parametrize("w_bits", [8, 4])
def test_encoder_block_is_the_chain_of_its_parts(orc, w_bits):
    shape = synth.BlockShape("tiny", 2, 21, 32, 2, 16, 64, True)
    spec = synth.make_block(shape, seed=3, w_bits=w_bits)
    d = _prepared_block(orc, spec)
    y = orc.encoder_block(spec.x, d)
    T, D = shape.T, shape.D
    h1 = orc.layernorm(spec.x, d["ln1_gamma"], d["ln1_beta"], d["ln1"])
    qkv = orc.linear(h1, d["w_qkv"], d["b_qkv"], d["m_qkv"], d["s_qkv"], w_bits=w_bits)
    to_heads = lambda a: np.ascontiguousarray(a.reshape(shape.B, shape.N, shape.H, shape.dh).transpose(0, 2, 1, 3))
    att = orc.attention_block(to_heads(qkv[:, :D]), to_heads(qkv[:, D:2 * D]), to_heads(qkv[:, 2 * D:]),
                              d["sm"], d["pv_rq"], d["attn_bias"], None).reshape(T, D)
    x1 = orc.linear(att, d["w_proj"], d["b_proj"], d["m_proj"], d["s_proj"], 0, spec.x, d["res1_rq"], w_bits=w_bits)
    h2 = orc.layernorm(x1, d["ln2_gamma"], d["ln2_beta"], d["ln2"])
    hid = orc.mlp_block(h2, d["w_fc1"], d["b_fc1"], d["m_fc1"], d["s_fc1"], d["gelu"], w_bits=w_bits)
    want = orc.linear(hid, d["w_fc2"], d["b_fc2"], d["m_fc2"], d["s_fc2"], 0, x1, d["res2_rq"], w_bits=w_bits)
    assert (y == want).all()
    # and the whole integer block tracks the fp64 computation it quantises (loose: W4 is coarse)
    assert np.abs(hid.astype(int)).max() > 20 and len(np.unique(y)) > 20


def test_encoder_block_w6a6_is_the_chain_of_its_parts(orc):
    """6-bit weights and activations (the W6A6 column of the object-detection results, Table 8): every tensor between two operators stays in
    the signed 6-bit range (residual stream included), and the block is the chain of the stand-alone operators
    run at that width."""
    from oracle import compose
    shape = synth.BlockShape("tiny", 2, 21, 32, 2, 16, 64, True)
    spec = synth.make_block(shape, seed=5, w_bits=6, a_bits=6)
    for lin in (spec.qkv, spec.proj, spec.fc1, spec.fc2):
        assert np.abs(lin.w.astype(int)).max() <= 31
    assert np.abs(spec.x.astype(int)).max() <= 32
    d = compose.block_params(spec, (0, 0, 0, 0))
    y = orc.encoder_block(spec.x, d)
    T, D = shape.T, shape.D
    h1 = orc.layernorm(spec.x, d["ln1_gamma"], d["ln1_beta"], d["ln1"])
    qkv = orc.linear(h1, d["w_qkv"], d["b_qkv"], d["m_qkv"], d["s_qkv"], out_bits=6)
    to_heads = lambda a: np.ascontiguousarray(a.reshape(shape.B, shape.N, shape.H, shape.dh).transpose(0, 2, 1, 3))
    att = orc.attention_block(to_heads(qkv[:, :D]), to_heads(qkv[:, D:2 * D]), to_heads(qkv[:, 2 * D:]),
                              d["sm"], d["pv_rq"], d["attn_bias"], None).reshape(T, D)
    x1 = orc.linear(att, d["w_proj"], d["b_proj"], d["m_proj"], d["s_proj"], d["proj_zp"], spec.x, d["res1_rq"],
                    out_bits=6)
    h2 = orc.layernorm(x1, d["ln2_gamma"], d["ln2_beta"], d["ln2"])
    hid = orc.mlp_block(h2, d["w_fc1"], d["b_fc1"], d["m_fc1"], d["s_fc1"], d["gelu"])
    want = orc.linear(hid, d["w_fc2"], d["b_fc2"], d["m_fc2"], d["s_fc2"], d["fc2_zp"], x1, d["res2_rq"], out_bits=6)
    for t in (h1, qkv, att, x1, h2, hid, want):
        assert t.min() >= -32 and t.max() <= 31
    assert (y == want).all()
    assert len(np.unique(y)) > 20 and len(np.unique(hid)) > 10


def test_mlp_block_fc1_epilogue(orc):
    rng = np.random.default_rng(13)
    M, D, Dh = 9, 32, 48
    x = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    w1 = rng.integers(-128, 128, size=(Dh, D)).astype(np.int8)
    b1 = rng.integers(-500, 500, size=Dh).astype(np.int32)
    m1, s1 = _prep_channels(orc, 2.0 ** rng.uniform(-6, -3, size=Dh))
    gc = orc.gelu_prepare(2e-3, 12, 0.03, -100, 8, 0)
    h = orc.mlp_block(x, w1, b1, m1, s1, gc)
    acc = x.astype(np.int64) @ w1.astype(np.int64).T + b1
    xin = np.clip(_np_requant_vec(acc, m1, s1), -2048, 2047).astype(np.int32)
    assert (h == orc.gelu(xin, gc)).all()
