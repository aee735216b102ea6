"""Data-aware refit of the quartic erf polynomial (Sec. 3.3, Eqs. (3)-(4)): pins of the oracle's fit and the
library's host-side fit against it.  CPU only (the fit and the constant preparation run on the host)."""
import math

import numpy as np
import pytest
from scipy.special import erf

from oracle import refit
from paper_2511_15369_b200 import api

PAPER_A, PAPER_B = -0.019913, -2.698088          # printed under Eq. (3)


def _ss(x, a, b):
    r = erf(x) - refit.erf_poly4(x, a, b)
    return float(np.dot(r, r))


def test_fit_recovers_known_coefficients():
    x = np.linspace(-4.0, 4.0, 2001)
    for a0, b0 in ((-0.0123, -3.1), (PAPER_A, PAPER_B), (-0.05, -2.0)):
        a, b, ss = refit.fit_to(x, refit.erf_poly4(x, a0, b0))
        assert a == pytest.approx(a0, abs=1e-10) and b == pytest.approx(b0, abs=1e-8) and ss < 1e-18


def test_fit_is_the_least_squares_optimum_on_the_papers_range():
    # Table 3 evaluates on (-3, 3): the refit on that grid cannot be worse than the printed coefficients,
    # and is a stationary point of the loss
    x = np.linspace(-3.0, 3.0, 4001)
    a, b, rms = refit.fit_erf_poly4(-3.0, 3.0, 4001)
    n = np.count_nonzero(x)
    assert math.sqrt(_ss(x, PAPER_A, PAPER_B) / n) == pytest.approx(0.0098, abs=5e-5)     # the paper's own error
    assert rms < 0.0098 and rms == pytest.approx(math.sqrt(_ss(x, a, b) / n), rel=1e-12)
    base = _ss(x, a, b)
    for da, db in ((1e-5, 0), (-1e-5, 0), (0, 1e-3), (0, -1e-3), (1e-5, 1e-3), (-1e-5, -1e-3)):
        assert _ss(x, a + da, b + db) > base
    # the optimum is close to the printed coefficients (which were fitted on image data, not on a uniform grid)
    assert abs(a - PAPER_A) < 1.0e-3 and abs(b - PAPER_B) < 0.03


def test_fit_depends_on_the_data_range():
    a1, b1, r1 = refit.fit_erf_poly4(-1.5, 1.5)
    a2, b2, r2 = refit.fit_erf_poly4(-6.0, 2.0)
    assert (a1, b1) != (a2, b2)
    x = np.linspace(-1.5, 1.5, 4001)
    assert _ss(x, a1, b1) < _ss(x, a2, b2) and _ss(x, a1, b1) < _ss(x, PAPER_A, PAPER_B)
    # symmetric in the sign of the range: both functions are odd
    a3, b3, _ = refit.fit_erf_poly4(-2.0, 6.0)
    assert a3 == pytest.approx(a2, abs=1e-9) and b3 == pytest.approx(b2, abs=1e-7)


@pytest.mark.parametrize("lo,hi,points", [(-3.0, 3.0, 4001), (-1.5, 1.5, 4001), (-6.0, 2.0, 1001), (0.5, 2.5, 513)])
def test_library_fit_matches_oracle(lo, hi, points):
    a, b, rms = api.gelu_fit(lo, hi, points)
    ao, bo, ro = refit.fit_erf_poly4(lo, hi, points)
    assert a == pytest.approx(ao, abs=1e-8) and b == pytest.approx(bo, abs=1e-6) and rms == pytest.approx(ro, rel=1e-8)
    assert a < 0 and b < 0


def test_prepare_with_coefficients(orc):
    for S, bits in ((1.3e-4, 16), (2e-3, 12), (0.05, 8)):
        for a, b in ((PAPER_A, PAPER_B), api.gelu_fit(-3, 3)[:2], (-0.0123, -3.1)):
            try:
                c = api.gelu_prepare_coeffs(S, bits, 0.02, -100, 8, a, b)
            except api.IptqError as e:                      # |b| / S' beyond 15 bits: both sides must refuse
                assert e.status == api.ERR_SCALE_RANGE
                with pytest.raises(orc.OracleError):
                    orc.gelu_prepare_coeffs(S, bits, 0.02, -100, 8, a, b)
                continue
            o = orc.gelu_prepare_coeffs(S, bits, 0.02, -100, 8, a, b)
            for f in ("variant", "in_bits", "Bq", "sh2", "C", "gs"):
                assert getattr(c, f) == getattr(o, f), (f, S, bits)
            assert (c.out.mult, c.out.shift, c.out.zp) == (o.out.mult, o.out.shift, o.out.zp)
        # the printed coefficients give the constants of the stock quartic variant
        c, d = api.gelu_prepare_coeffs(S, bits, 0.02, -100, 8, PAPER_A, PAPER_B), api.gelu_prepare(S, bits, 0.02, -100, 8, 0)
        assert (c.Bq, c.sh2, c.C, c.gs) == (d.Bq, d.sh2, d.C, d.gs)
    with pytest.raises(api.IptqError):
        api.gelu_prepare_coeffs(1e-3, 16, 0.02, 0, 8, 0.02, -2.7)
    with pytest.raises(orc.OracleError):
        orc.gelu_prepare_coeffs(1e-3, 16, 0.02, 0, 8, -0.02, 2.7)
    assert api.lib().iptq_gelu_fit(1.0, 1.0, 100, None, None, None) == api.ERR_NULL


def test_refitted_gelu_tracks_the_float_gelu(orc):
    """Integer GELU with refitted coefficients against fp64 GELU on the range it was fitted for."""
    lo, hi, bits = -2.0, 2.0, 14
    S = 2.0 / 8191
    a, b, _ = refit.fit_erf_poly4(lo / math.sqrt(2), hi / math.sqrt(2))      # the polynomial sees x / sqrt 2
    x = np.arange(-8191, 8192, 3, dtype=np.int64)
    ref = 0.5 * (x * S) * (1.0 + erf(x * S / math.sqrt(2)))
    errs = {}
    for name, c in (("fit", orc.gelu_prepare_coeffs(S, bits, 0.02, 0, 8, a, b)), ("paper", orc.gelu_prepare(S, bits, 0.02, 0, 8, 0))):
        y = np.array([orc.gelu_core(int(v), c) for v in x], dtype=np.float64) * orc.gelu_core_scale(S, c)
        errs[name] = float(np.sqrt(np.mean((y - ref) ** 2)))
    assert errs["fit"] < 0.012 and errs["paper"] < 0.012
