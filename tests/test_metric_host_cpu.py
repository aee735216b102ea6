"""Host side of the Unified Metric in the library (Softplus, SQNR, the term of Eq. (16), operation counts, the
selection) against the oracle.  No GPU: these entry points run on the host."""
import math

import numpy as np
import pytest

from oracle import metric
from paper_2511_15369_b200 import api


def test_softplus_and_sqnr_match_oracle():
    for v in list(np.linspace(-50, 50, 201)) + [-800.0, 800.0, 1e6, -1e6, 0.0]:
        assert api.softplus(v) == pytest.approx(metric.softplus(v), rel=1e-15, abs=1e-300)
    assert api.sqnr_db(1e4, 100.0) == pytest.approx(20.0, abs=1e-12)          # worked example beside Eq. (18)
    assert 22.21 <= api.sqnr_db(1e4, 60.0) < 22.22
    assert api.sqnr_db(3.0, 0.0) == math.inf
    rng = np.random.default_rng(0)
    for a, b in rng.uniform(1e-9, 1e9, size=(100, 2)):
        assert api.sqnr_db(a, b) == pytest.approx(metric.sqnr_db(a, b), rel=1e-14, abs=1e-12)


def test_metric_term_matches_oracle():
    rng = np.random.default_rng(1)
    for _ in range(300):
        q = rng.uniform(-10, 80)
        p = 10.0 ** rng.uniform(-6, 3)
        c = 10.0 ** rng.uniform(3, 9)
        unit = 10.0 ** rng.integers(0, 8)
        assert api.metric_term(q, p, c, unit) == pytest.approx(metric.layer_term(q, p, c, unit), rel=1e-14)
    assert api.metric_term(math.inf, 0.0, 1e6, 1e6) == pytest.approx(metric.layer_term(math.inf, 0.0, 1e6, 1e6), rel=1e-15)
    assert api.metric_term(math.log(math.expm1(1 / math.log(2))), 0.0, 0.0, 1.0) == pytest.approx(1 / math.log(2), rel=1e-14)


def test_op_counts_and_selection_match_oracle():
    for kind in (0, 1, 2):
        for v in (0, 1, 2, 3) if kind == 0 else (0, 1, 2):
            for rows, n in ((1, 1), (197, 197), (9456, 197), (1576, 3072), (0, 64)):
                assert api.op_count(kind, v, rows, n) == metric.op_count(kind, v, rows, n)
    assert api.op_count(3, 0, 1, 1) < 0 and api.op_count(0, 4, 1, 1) < 0 and api.op_count(1, 3, 1, 1) < 0 and api.op_count(0, -1, 1, 1) < 0
    rng = np.random.default_rng(2)
    for _ in range(50):
        t = list(rng.integers(0, 4, size=rng.integers(1, 6)) / 4.0)
        assert api.metric_select(t) == metric.select(t)
    assert api.lib().iptq_metric_select(None, 0) == -1
