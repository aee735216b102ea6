"""CPU oracle of the Unified Metric for approximation-function assignment (Sec. 3.5, Eqs. (16)-(20)).

TEST INFRASTRUCTURE ONLY: plain numpy in fp64, one formula per function, written from the paper's equations.
It shares nothing with the CUDA library; only tests, the smoke check and the benchmark's CPU legs may import it.

For one activation layer and one candidate approximation function the paper compares the full-precision
output X of the layer with the de-quantised output Q of the integer function on the same input:

    Q (sensitivity)  = SQNR in dB                      Eq. (18)
    P (perturbation) = || X - Q ||_2^2                 Eq. (19)
    C (cost)         = integer operation count         Eq. (20)
    N(v)             = log(1 + exp(v))   (Softplus)    Eq. (17)
    Omega            = sum over layers of  3 / ( 1/N(Q) + N(P) + N(C) )      Eq. (16)

and assigns to every layer the candidate with the largest term (Sec. 3.5, stage 2 of the pipeline figure).

Readings (the paper is silent or inconsistent here):
  * Eq. (18) is printed as "20 log" of a ratio of powers, but the worked example beside it (signal power 1e4,
    noise 100 -> 20 dB, noise 60 -> 22.21 dB) is 10 log10 of that ratio: the example decides.
  * X is the float function evaluated on the de-quantised integer input (scale * integer), so that X and Q differ
    only by what the integer function and its output quantiser add.
  * LayerNorm reference: biased variance, no epsilon; a constant row maps to beta.
  * Units of P and C: P is the plain sum of squared differences over the tensor handed in; C is handed to N()
    after division by ``c_unit`` operations (default 1e6: mega-operations) -- raw counts of 1e7..1e9 would make
    N(C) the only term that matters.  Both are parameters, not facts from the paper.
  * The operation counts themselves (``op_count``) follow this library's integer definitions, one count per
    add / subtract / multiply / shift / compare / divide, "counting as in FLOPs" (Sec. 3.5).  The paper prints
    no counts: parity unpinned for C.
"""
from __future__ import annotations

import math

import numpy as np

SOFTMAX, GELU, LAYERNORM = 0, 1, 2


# ------------------------------------------------------------------ Eqs. (17)-(19), (16)

def softplus(v: float) -> float:
    """Eq. (17), N(v) = log(1 + exp(v)), evaluated without overflow."""
    v = float(v)
    return max(v, 0.0) + math.log1p(math.exp(-abs(v)))


def sqnr_db(sum_x2: float, sum_err2: float) -> float:
    """Eq. (18) in the reading the worked example fixes: 10 log10(E[X^2] / E[(X - Q)^2]).  Both expectations are
    over the same elements, so the ratio of the sums is the ratio of the means."""
    if sum_err2 == 0.0:
        return math.inf
    return 10.0 * math.log10(sum_x2 / sum_err2)


def layer_term(q_db: float, p: float, c_ops: float, c_unit: float = 1.0e6) -> float:
    """One summand of Eq. (16): three over the sum of the reciprocal-form factors."""
    nq = softplus(q_db)
    inv_nq = 0.0 if math.isinf(nq) else 1.0 / nq
    return 3.0 / (inv_nq + softplus(p) + softplus(c_ops / c_unit))


def unified_metric(terms) -> float:
    """Eq. (16): sum of the per-layer terms."""
    return float(math.fsum(terms))


def error_sums(x_ref: np.ndarray, q_deq: np.ndarray):
    """(sum X^2, sum (X - Q)^2) in extended precision."""
    x = np.asarray(x_ref, dtype=np.longdouble).ravel()
    d = x - np.asarray(q_deq, dtype=np.longdouble).ravel()
    return float(np.sum(x * x)), float(np.sum(d * d))


# ------------------------------------------------------------------ float layers (X)

def softmax_float(scores: np.ndarray, in_scale: float) -> np.ndarray:
    z = np.asarray(scores, dtype=np.float64) * in_scale
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def gelu_float(x: np.ndarray, in_scale: float) -> np.ndarray:
    from scipy.special import erf
    v = np.asarray(x, dtype=np.float64) * in_scale
    return 0.5 * v * (1.0 + erf(v / math.sqrt(2.0)))


def layernorm_float(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, ptf_shift: np.ndarray | None = None) -> np.ndarray:
    v = np.asarray(x, dtype=np.float64)
    if ptf_shift is not None:
        v = v * np.exp2(np.asarray(ptf_shift, dtype=np.float64))      # power-of-two factor per channel
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    sd = np.sqrt(var)
    g = np.asarray(gamma, dtype=np.float64)
    b = np.asarray(beta, dtype=np.float64)
    with np.errstate(invalid="ignore", divide="ignore"):
        y = (v - mu) / sd * g + b
    return np.where(sd == 0.0, np.broadcast_to(b, v.shape), y)


# ------------------------------------------------------------------ de-quantised integer layers (Q)

def softmax_deq(probs: np.ndarray, out_bits: int) -> np.ndarray:
    return np.asarray(probs, dtype=np.float64) / float(1 << (out_bits - 1))


def log2_deq(codes: np.ndarray) -> np.ndarray:
    """Logarithm candidate: probability 2^-code for codes 0..15, 0 for the "zero" code 255."""
    c = np.asarray(codes)
    return np.where(c == 255, 0.0, np.exp2(-np.minimum(c, 15).astype(np.float64)))


def affine_deq(y: np.ndarray, out_scale: float, out_zp: int) -> np.ndarray:
    return (np.asarray(y, dtype=np.float64) - float(out_zp)) * out_scale


# ------------------------------------------------------------------ Eq. (20): operation counts (this library's reading)

# Counted mechanically: one per binary add / subtract / multiply / divide / shift / mask and per comparison (min, max,
# |.|, sign and leading-one position are one each); sign flips, copies, constants prepared before inference and
# values that do not change inside a row (counted once per row) are not per-element operations.
_SOFTMAX_PER_ELEM = {0: 21, 1: 17, 2: 15, 3: 25}     # SM_BITEXP, SM_SHIFTMAX, SM_POLY, SM_LOG2
_SOFTMAX_PER_ROW = {0: 1, 1: 1, 2: 1, 3: 1}          # the division of Eq. (15); logarithm candidate: twice the row sum
_GELU_PER_ELEM = {0: 21, 1: 20, 2: 34}               # GELU_POLY4, GELU_POLY2, GELU_SHIFT
_LN_PER_ELEM = {0: 16, 1: 16, 2: 17}                 # LN_SHIFT, LN_NEWTON, LN_PTF (one more shift per element)
LN_NEWTON_NOMINAL_STEPS = 5                          # most steps the iterated square root takes on LayerNorm rows of the workload
_LN_PER_ROW = {0: 38, 1: 28, 2: 28}                  # variance 3, start value 4, steps (10 x 3 / 5 x 4), reciprocal 1


def op_count(kind: int, variant: int, rows: int, row_len: int) -> float:
    """Integer operations of one layer on a [rows, row_len] tensor (GELU: rows * row_len elements).

    Softmax, per element: running max 1, distance 1, clamp 1, Eq. (7) 4, Eq. (8) 3 (divide, multiply, subtract),
    Phi + x0 6 (Bit-exp; 2 for Shiftmax), Eq. (9) 2, sum 1, Eq. (15) 2; one division per row.  Second-order
    polynomial exponential: max 1, distance 1, clamp 1, octave divide 1, remainder 2, polynomial 3, normalise 2,
    octave shift 1, sum 1, Eq. (15) 2.  Logarithm candidate: the same exponential and sum (13), zero test 1,
    round(sum / e) 3 (twice the sum once per row), leading-one position 2, rounding bit 5, range test 1.
    GELU, per element: clamp 2, |x| 1, min 1, subtract 1, square 1, shift 1, second square 1 (fourth order only),
    C - (.) 1, sign 1, times E 1, + C 1, shift 1, x * G 1, requantise 7 (multiply, high word, round, shift, zero
    point, two clamps).  Shift-based sigmoid form: clamp 2, 1.702 x by shifts 6, |.| and clamp 2, exponential 11,
    D + e 1, divide 1, select 1, multiply 1, shift 1, x * sigma 1, requantise 7.
    LayerNorm, per element: sum 1, square-and-add 2, D x - sum 2, times reciprocal and shift 2, gamma/beta 2,
    requantise 7 (the power-of-two-factor variant shifts the input first: 1 more); per row: variance 3, start
    value of the square root 4, steps of the recurrence (divide, add, shift: 10 in the fixed-step variant; with
    the comparison that ends the iteration, 5 steps when iterated to convergence) and one reciprocal.
    """
    n = float(rows) * float(row_len)
    if kind == SOFTMAX:
        return _SOFTMAX_PER_ELEM[variant] * n + _SOFTMAX_PER_ROW[variant] * float(rows)
    if kind == GELU:
        return _GELU_PER_ELEM[variant] * n
    if kind == LAYERNORM:
        return _LN_PER_ELEM[variant] * n + _LN_PER_ROW[variant] * float(rows)
    raise ValueError("unknown layer kind")


# ------------------------------------------------------------------ stage 1 / stage 2 on one layer

def evaluate(x_ref: np.ndarray, q_deq: np.ndarray, c_ops: float, c_unit: float = 1.0e6):
    """Returns (Q in dB, P, term of Eq. (16)) for one candidate."""
    sx2, se2 = error_sums(x_ref, q_deq)
    q = sqnr_db(sx2, se2)
    return q, se2, layer_term(q, se2, c_ops, c_unit)


def select(terms) -> int:
    """Stage 2: index of the largest term; the first one wins a tie."""
    best = 0
    for i, t in enumerate(terms):
        if t > terms[best]:
            best = i
    return best
