"""CPU oracle of the data-aware refit of the quartic erf polynomial (Sec. 3.3, Eqs. (3)-(4)).

TEST INFRASTRUCTURE ONLY.  The paper re-computes the coefficients (a, b) of

    L(x; a, b) = sign(x) * ( a * (min(|x|, -b) + b)^4 + 1 )                       Eq. (3)

for the value range of the data, [min(T), max(T)], by least squares against erf (Eq. (4)):

    argmin_{a, b}  sum_i ( erf(x_i) - L(x_i; a, b) )^2 ,   x_i in [min(T), max(T)].

Reading: the x_i are a uniform grid over that range (the paper gives the range, not the sample).  For a fixed b
the problem is linear in a, so a(b) has a closed form and the search is one-dimensional in b.
"""
from __future__ import annotations

import math

import numpy as np


def erf_poly4(x, a: float, b: float):
    """Eq. (3)."""
    x = np.asarray(x, dtype=np.float64)
    return np.sign(x) * (a * (np.minimum(np.abs(x), -b) + b) ** 4 + 1.0)


def _a_of_b(u, target, b):
    t = (np.minimum(u, -b) + b) ** 4
    den = float(np.dot(t, t))
    return float(np.dot(t, target - 1.0)) / den if den > 0.0 else 0.0


def fit_to(x, target, b_lo: float = -8.0, b_hi: float = -0.25):
    """Least-squares (a, b) of Eq. (3) against ``target`` on the points x (odd symmetry: both are folded to
    |x|).  Returns (a, b, sum of squared residuals)."""
    x = np.asarray(x, dtype=np.float64)
    u = np.abs(x)
    tgt = np.sign(x) * np.asarray(target, dtype=np.float64)       # odd target folded to the positive side
    keep = x != 0.0
    u, tgt = u[keep], tgt[keep]

    def loss(b):
        a = _a_of_b(u, tgt, b)
        r = tgt - (a * (np.minimum(u, -b) + b) ** 4 + 1.0)
        return float(np.dot(r, r))

    # coarse scan, then golden section around the best cell
    grid = np.linspace(b_lo, b_hi, 311)
    k = int(np.argmin([loss(b) for b in grid]))
    lo, hi = grid[max(k - 1, 0)], grid[min(k + 1, len(grid) - 1)]
    g = (math.sqrt(5.0) - 1.0) / 2.0
    c, d = hi - g * (hi - lo), lo + g * (hi - lo)
    fc, fd = loss(c), loss(d)
    for _ in range(200):
        if fc < fd:
            hi, d, fd = d, c, fc
            c = hi - g * (hi - lo)
            fc = loss(c)
        else:
            lo, c, fc = c, d, fd
            d = lo + g * (hi - lo)
            fd = loss(d)
        if hi - lo < 1e-12:
            break
    b = 0.5 * (lo + hi)
    return _a_of_b(u, tgt, b), b, loss(b)


def fit_erf_poly4(lo: float, hi: float, points: int = 4001):
    """Eq. (4) on a uniform grid over [lo, hi].  Returns (a, b, rms residual)."""
    from scipy.special import erf
    x = np.linspace(lo, hi, points)
    a, b, ss = fit_to(x, erf(x))
    return a, b, math.sqrt(ss / np.count_nonzero(x))
