"""Pins the operation counts of Eq. (20) (Sec. 3.5: the complexity term counts arithmetic and bit operations of a
layer) mechanically: every oracle function is written out once more on an integer type that counts each binary
add / subtract / multiply / divide / shift / mask, each comparison (min, max, |.|, sign and leading-one position
are one comparison-like operation each), and the tables of ``oracle.metric.op_count`` must equal the counted
totals for one element and one row of every variant.  Not counted: sign flips, copies, the selection that follows
a counted comparison, constants prepared before inference, and guards that only exist because C shifts are
undefined for large counts.  An entry that is off by one fails here."""
import numpy as np
import pytest

import oracle
from oracle import metric as om
from paper_2511_15369_b200 import synth


class Counter:
    def __init__(self):
        self.n = 0


class CI:
    """Integer that counts the operations applied to it (shared counter)."""
    __slots__ = ("v", "c")

    def __init__(self, v, c):
        self.v, self.c = int(v), c

    def _o(self, other):
        return other.v if isinstance(other, CI) else int(other)

    def _bin(self, other, f):
        self.c.n += 1
        return CI(f(self.v, self._o(other)), self.c)

    def __add__(self, o): return self._bin(o, lambda a, b: a + b)
    def __radd__(self, o): return self._bin(o, lambda a, b: b + a)
    def __sub__(self, o): return self._bin(o, lambda a, b: a - b)
    def __rsub__(self, o): return self._bin(o, lambda a, b: b - a)
    def __mul__(self, o): return self._bin(o, lambda a, b: a * b)
    def __rmul__(self, o): return self._bin(o, lambda a, b: b * a)
    def __floordiv__(self, o): return self._bin(o, lambda a, b: a // b)
    def __rfloordiv__(self, o): return self._bin(o, lambda a, b: b // a)
    def __lshift__(self, o): return self._bin(o, lambda a, b: a << b)
    def __rlshift__(self, o): return self._bin(o, lambda a, b: b << a)
    def __rshift__(self, o): return self._bin(o, lambda a, b: a >> b)       # Python's >> floors, as the oracle's fshr
    def __and__(self, o): return self._bin(o, lambda a, b: a & b)
    def __neg__(self): return CI(-self.v, self.c)                           # a sign flip is not an operation

    def _cmp(self, o, f):
        self.c.n += 1
        return f(self.v, self._o(o))

    def __lt__(self, o): return self._cmp(o, lambda a, b: a < b)
    def __le__(self, o): return self._cmp(o, lambda a, b: a <= b)
    def __gt__(self, o): return self._cmp(o, lambda a, b: a > b)
    def __ge__(self, o): return self._cmp(o, lambda a, b: a >= b)
    def __eq__(self, o): return self._cmp(o, lambda a, b: a == b)
    def __ne__(self, o): return self._cmp(o, lambda a, b: a != b)
    def __hash__(self): return hash(self.v)


def _val(a):
    return a.v if isinstance(a, CI) else int(a)


def cmin(a, b):
    c = a.c if isinstance(a, CI) else b.c
    c.n += 1                                  # one comparison
    return CI(min(_val(a), _val(b)), c)


def cmax(a, b):
    c = a.c if isinstance(a, CI) else b.c
    c.n += 1
    return CI(max(_val(a), _val(b)), c)


def cabs(a):
    a.c.n += 1                                # one comparison-like operation
    return CI(abs(a.v), a.c)


def csign(a):
    a.c.n += 1
    return CI((a.v > 0) - (a.v < 0), a.c)


def cbitlen(a):
    a.c.n += 1                                # leading-one position
    return CI(a.v.bit_length(), a.c)


def requant(y, rq):
    """R: hi32 of the product, round half up, shift, zero point, clamp (two comparisons)."""
    hi = (y * rq.mult) >> 32
    v = ((hi + (1 << (rq.shift - 1))) >> rq.shift) + rq.zp
    return cmin(cmax(v, rq.qmin), rq.qmax)


# ------------------------------------------------------------------ Softmax (Sec. 3.4)

def softmax_exp(d, c):
    if c.variant in (2, 3):                               # second-order polynomial exponential
        z = d // c.qln2
        p = -(d - z * c.qln2)
        t = p + c.qb
        poly = t * t + c.qc
        return ((poly << c.norm_l) >> c.norm_r) >> z
    Qd = -d
    Qp = Qd + (Qd >> 1) - (Qd >> 4)                       # Eq. (7)
    P = -Qp
    q = P // c.x0                                         # Eq. (8)
    r = P - q * c.x0
    u = -r
    base = (u >> 1) + (u >> 3) + (u >> 4) + c.x0 if c.variant == 0 else (u >> 1) + c.x0   # Eqs. (13)-(14) / (10)
    return (base << c.nsh) >> q                           # Eq. (9)


def softmax_row_counts(scores, c):
    """(operations of every element, operations per row, outputs) of one Softmax row.  Loop-invariant values
    (the row's division, twice the row sum) count once per row."""
    n = len(scores)
    cnts = [Counter() for _ in range(n)]
    row = Counter()
    s = [CI(v, cnts[j]) for j, v in enumerate(scores)]
    # Eq. (6): running maximum, one comparison per element
    mx = scores[0]
    for j in range(n):
        mx = cmax(s[j], mx).v
    e, total = [], 0
    for j in range(n):
        d = cmin(mx - s[j], c.dcap)
        e.append(softmax_exp(d, c))
        total = (e[-1] + total).v                          # the running sum: one addition per element
    out = []
    if c.variant == 3:
        two_sum = (2 * CI(total, row)).v
        for j in range(n):
            if e[j] == 0:
                out.append(255)
                continue
            r = (two_sum + e[j]) // (2 * e[j])             # round(sum / e), halves up
            fl = cbitlen(r) - 1
            code = fl
            if fl >= 1:
                code = fl + ((r >> (fl - 1)) & 1)
            out.append(255 if code > 15 else code.v)
        return [k.n for k in cnts], row.n, out
    f = ((1 << c.M) // CI(total, row)).v                   # Eq. (15): one division per row
    sh = c.M - (c.out_bits - 1)
    for j in range(n):
        out.append(((f * e[j]) >> sh).v)
    return [k.n for k in cnts], row.n, out


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
def test_softmax_counts(variant):
    n = 197
    c = oracle.softmax_prepare(synth.SOFTMAX_SCALE_ACC, n, 4 if variant == 3 else 8, variant)
    s = synth.quantize_scores(synth.softmax_logits(2, n, seed=5), synth.SOFTMAX_SCALE_ACC)
    counts, per_row, out = softmax_row_counts(s[0].tolist(), c)
    assert out == oracle.softmax(s[:1], c)[0].tolist()     # the transcription computes what the oracle computes
    # the layer's count is that of an element that takes every step (the logarithm candidate skips the rounding
    # for entries whose exponential is 0 or whose ratio is 1)
    assert max(counts) == om._SOFTMAX_PER_ELEM[variant], (variant, max(counts))
    if variant != 3:
        assert min(counts) == max(counts)
    assert per_row == om._SOFTMAX_PER_ROW[variant] == 1
    assert om.op_count(om.SOFTMAX, variant, 7, n) == 7 * n * max(counts) + 7 * per_row


# ------------------------------------------------------------------ GELU (Sec. 3.3)

def gelu_elem(xv, c, cnt):
    x = CI(xv, cnt)
    lo, hi = -(1 << (c.in_bits - 1)), (1 << (c.in_bits - 1)) - 1
    x = cmin(cmax(x, lo), hi)
    if c.variant == 2:
        xp = x + (x >> 1) + (x >> 3) + (x >> 4)
        d = cmin(cabs(xp), c.dcap)
        Qd = -d
        Qp = Qd + (Qd >> 1) - (Qd >> 4)
        P = -Qp
        q = P // c.x0
        r = P - q * c.x0
        e = ((((-r) >> 1) + c.x0) << c.nsh) >> q
        D = int(c.x0) << int(c.nsh)                        # a constant
        f = (1 << 31) // (D + e)
        cnt.n += 1                                         # the test xp >= 0 that picks the numerator
        num = D if xp.v >= 0 else e
        sig = (f * num) >> 16
        y = x * sig
    else:
        m = cmin(cabs(x), c.Bq)
        t = c.Bq - m
        t2 = (t * t) >> c.sh2
        pw = t2 * t2 if c.variant == 0 else t2
        E = c.C - pw
        G = csign(x) * E + c.C
        y = x * (G >> c.gs)
    return requant(y, c.out).v


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_gelu_counts(variant):
    bits, S = (16, 1.3e-4) if variant != 2 else (12, 0.003)
    c = oracle.gelu_prepare(S, bits, 0.03, -7, 8, variant)
    xs = np.array([-30000, -4001, -1, 0, 3, 1777, 29000], dtype=np.int32)
    want = oracle.gelu(xs, c)
    counts = set()
    for xv, w in zip(xs.tolist(), want.tolist()):
        cnt = Counter()
        assert gelu_elem(xv, c, cnt) == w
        counts.add(cnt.n)
    assert counts == {om._GELU_PER_ELEM[variant]}, (variant, counts)
    assert om.op_count(om.GELU, variant, 3, 5) == 15 * om._GELU_PER_ELEM[variant]


# ------------------------------------------------------------------ LayerNorm

def isqrt_steps(V, variant, cnt):
    """The square-root recurrence on a counting integer; returns (root, steps run)."""
    Vc = CI(V, cnt)
    r = 1 << ((cbitlen(Vc) + 1) >> 1)
    if variant == 0:
        for _ in range(10):
            r = (r + Vc // r) >> 1
        return r, 10
    steps = 0
    while True:
        r1 = (r + Vc // r) >> 1
        steps += 1
        if r1 >= r:
            return r, steps
        r = r1


def layernorm_row_counts(x, gq, bq, ptf, c):
    cnt = Counter()
    D = len(x)
    xs = [CI(v, cnt) for v in x]
    s1, s2 = CI(0, cnt), CI(0, cnt)
    xh = []
    for j in range(D):
        h = xs[j] << int(ptf[j]) if ptf is not None else xs[j]
        xh.append(h)
        s1 = s1 + h
        s2 = s2 + h * h
    elem_ops = cnt.n
    V = D * s2 - s1 * s1
    r, steps = isqrt_steps(V.v, c.variant, cnt) if V.v else (CI(0, cnt), 0)
    F = (1 << 40) // r
    row_ops = cnt.n - elem_ops
    cnt.n = elem_ops
    out = []
    for j in range(D):
        u = D * xh[j] - s1
        nq = (u * F) >> 30
        v = nq * int(gq[j]) + int(bq[j])
        out.append(requant(v, c.out).v)
    return cnt.n / D, row_ops, steps, out


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_layernorm_counts(variant):
    xf, gamma, beta, _ = synth.ln_values(64, 192, seed=0)
    xq, _ = synth.quantize_sym(xf, 8, np.int8)
    So, zp = synth.affine_out_quant(synth.layernorm_ref(xq.astype(np.float64), gamma, beta))
    gq, bq, c = oracle.layernorm_prepare(gamma, beta, So, zp, 8, variant)
    ptf = (np.arange(192) % 4).astype(np.uint8) if variant == 2 else None
    want = oracle.layernorm(xq, gq, bq, c, ptf)
    most_steps = 0
    for i in range(xq.shape[0]):
        per_elem, per_row, steps, out = layernorm_row_counts(xq[i].tolist(), gq, bq, ptf, c)
        assert out == want[i].tolist()
        assert per_elem == om._LN_PER_ELEM[variant], (variant, per_elem)
        if variant == 0:
            assert per_row == om._LN_PER_ROW[0], per_row
        else:
            # iterated to convergence: the table holds the count at the nominal number of steps, which the
            # rows of this workload never exceed; one step is a division, an addition, a shift and the comparison
            # that ends the loop
            assert per_row == om._LN_PER_ROW[variant] - 4 * (om.LN_NEWTON_NOMINAL_STEPS - steps), (per_row, steps)
            most_steps = max(most_steps, steps)
    if variant != 0:
        assert most_steps == om.LN_NEWTON_NOMINAL_STEPS
    assert om.op_count(om.LAYERNORM, variant, 4, 192) == 4 * 192 * om._LN_PER_ELEM[variant] + 4 * om._LN_PER_ROW[variant]


def test_library_table_equals_the_oracle_table():
    """The C-ABI library reports the same counts (host function: runs without a device)."""
    from paper_2511_15369_b200 import api
    for kind, variants in ((om.SOFTMAX, 4), (om.GELU, 3), (om.LAYERNORM, 3)):
        for v in range(variants):
            for rows, n in ((1, 1), (591, 197), (12608, 384)):
                assert api.op_count(kind, v, rows, n) == om.op_count(kind, v, rows, n), (kind, v, rows, n)
