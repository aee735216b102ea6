"""GPU parity of the Unified-Metric reductions and of the assignment driver (Sec. 3.5, Eqs. (16)-(20)) against the
numpy oracle on the same seeded inputs, through the C-ABI.

Tolerance: the sums are fp64 on both sides.  The device adds in a fixed tree order, the oracle in extended
precision; exp / erf / sqrt differ by at most a few units in the last place between the two math libraries, which
moves (X - Q)^2 by about 1e-13 relative when the error is a thousandth of the signal.  1e-9 relative on each sum
leaves four orders of margin and still catches any wrong element (one element of 10^5 contributes 1e-5)."""
import math

import numpy as np
import pytest

from paper_2511_15369_b200 import synth

pytestmark = pytest.mark.gpu
REL = 1e-9


@pytest.fixture(scope="module")
def api():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2511_15369_b200 import api as _api
    _api.lib()
    return _api


@pytest.fixture(scope="module")
def metric():
    from oracle import metric as m
    return m


def _cu(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _close(got, want):
    return all(abs(g - w) <= REL * abs(w) for g, w in zip(got, want))


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("rows,n", [(591, 197), (1000, 49), (33, 1), (9, 1000), (4099, 64)])
def test_metric_softmax_parity(api, orc, metric, variant, rows, n):
    S = synth.SOFTMAX_SCALE_ACC
    s = synth.quantize_scores(synth.softmax_logits(rows, n, seed=rows + n), S)
    p = orc.softmax(s, orc.softmax_prepare(S, n, 8, variant))
    want = metric.error_sums(metric.softmax_float(s, S), metric.softmax_deq(p, 8))
    sd = _cu(s)
    pd = api.softmax(sd, api.softmax_prepare(S, n, 8, variant))
    assert (pd.cpu().numpy() == p).all()
    got = api.metric_softmax(sd, pd, S, 8).cpu().numpy()
    assert _close(got, want), (got, want)
    assert n == 1 or (want[1] > 0 and want[0] > want[1])


@pytest.mark.parametrize("rows,n,scale", [(591, 197, synth.SOFTMAX_SCALE_ACC), (1000, 49, 1.0 / 700), (33, 1, 3e-4),
                                          (300, 197, synth.SOFTMAX_SCALE_8BIT)])
def test_metric_softmax_log2_candidate(api, orc, metric, rows, n, scale):
    s = synth.quantize_scores(synth.softmax_logits(rows, n, seed=rows), scale)
    codes = orc.softmax(s, orc.softmax_prepare(scale, n, 4, orc.SM_LOG2))
    want = metric.error_sums(metric.softmax_float(s, scale), metric.log2_deq(codes))
    sd = _cu(s)
    cd = api.softmax(sd, api.softmax_prepare(scale, n, 4, api.SM_LOG2))
    assert (cd.cpu().numpy() == codes).all()
    got = api.metric_softmax(sd, cd, scale, api.PROBS_LOG2).cpu().numpy()
    assert _close(got, want), (got, want)


@pytest.mark.parametrize("out_bits", [8, 6, 4])
def test_metric_softmax_out_bits_and_determinism(api, orc, metric, out_bits):
    S, rows, n = synth.SOFTMAX_SCALE_8BIT, 700, 197
    s = synth.quantize_scores(synth.softmax_logits(rows, n, seed=3), S)
    p = orc.softmax(s, orc.softmax_prepare(S, n, out_bits, 0))
    want = metric.error_sums(metric.softmax_float(s, S), metric.softmax_deq(p, out_bits))
    sd, pd = _cu(s), _cu(p)
    a = api.metric_softmax(sd, pd, S, out_bits).cpu().numpy()
    b = api.metric_softmax(sd, pd, S, out_bits).cpu().numpy()
    assert _close(a, want)
    assert a.tobytes() == b.tobytes()                     # fixed summation order


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("n", [151296, 4099, 3])
def test_metric_gelu_parity(api, orc, metric, variant, n):
    bits = 16 if variant != 2 else 12
    xall, S = synth.quantize_sym(synth.gelu_values(max(n, 4096), seed=n), bits)
    x = np.ascontiguousarray(xall[:n])
    So, zp = synth.affine_out_quant(synth.gelu_ref(xall[:4096] * S))
    y = orc.gelu(x, orc.gelu_prepare(S, bits, So, zp, 8, variant))
    want = metric.error_sums(metric.gelu_float(x, S), metric.affine_deq(y, So, zp))
    xd = _cu(x)
    yd = api.gelu(xd, api.gelu_prepare(S, bits, So, zp, 8, variant))
    assert (yd.cpu().numpy() == y).all()
    got = api.metric_gelu(xd, yd, S, So, zp).cpu().numpy()
    assert _close(got, want), (got, want)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("rows,dim", [(197, 192), (300, 384), (100, 768), (513, 96), (3, 3072), (5, 8)])
def test_metric_layernorm_parity(api, orc, metric, variant, rows, dim):
    xf, gamma, beta, _ = synth.ln_values(rows, dim, seed=dim)
    xq, _ = synth.quantize_sym(xf, 8, np.int8)
    xq[rows // 2] = 9                                     # a constant row: the float layer returns beta
    ptf = synth.ptf_shifts(xq) if variant == 2 else None
    So, zp = synth.affine_out_quant(synth.layernorm_ref(xq[:64].astype(np.float64), gamma, beta))
    gq, bq, co = orc.layernorm_prepare(gamma, beta, So, zp, 8, variant)
    y = orc.layernorm(xq, gq, bq, co, ptf)
    want = metric.error_sums(metric.layernorm_float(xq, gamma, beta, ptf), metric.affine_deq(y, So, zp))
    got = api.metric_layernorm(_cu(xq), _cu(y), _cu(gamma), _cu(beta), So, zp,
                               None if ptf is None else _cu(ptf)).cpu().numpy()
    assert _close(got, want), (got, want)


def test_metric_empty_inputs_and_errors(api):
    import torch
    dev = "cuda"
    z = api.metric_softmax(torch.empty((0, 197), dtype=torch.int32, device=dev),
                           torch.empty((0, 197), dtype=torch.uint8, device=dev), 3e-4).cpu().numpy()
    assert z.tolist() == [0.0, 0.0]
    z = api.metric_gelu(torch.empty(0, dtype=torch.int32, device=dev), torch.empty(0, dtype=torch.int8, device=dev),
                        1e-3, 0.03, 0).cpu().numpy()
    assert z.tolist() == [0.0, 0.0]
    g = torch.ones(96, dtype=torch.float32, device=dev)
    z = api.metric_layernorm(torch.empty((0, 96), dtype=torch.int8, device=dev),
                             torch.empty((0, 96), dtype=torch.int8, device=dev), g, g, 0.03, 0).cpu().numpy()
    assert z.tolist() == [0.0, 0.0]
    sc = api.MetricScratch(dev)
    s = torch.zeros((4, 8), dtype=torch.int32, device=dev)
    p = torch.zeros((4, 8), dtype=torch.uint8, device=dev)
    L = api.lib()
    assert L.iptq_metric_softmax(s.data_ptr(), p.data_ptr(), 4, 8, 3e-4, 8, None, sc.work.data_ptr(), None) == api.ERR_NULL
    assert L.iptq_metric_softmax(s.data_ptr(), p.data_ptr(), 4, 8, 3e-4, 8, sc.sums.data_ptr() + 8, sc.work.data_ptr(), None) == api.ERR_ALIGN
    assert L.iptq_metric_softmax(s.data_ptr(), p.data_ptr(), 4, 2000, 3e-4, 8, sc.sums.data_ptr(), sc.work.data_ptr(), None) == api.ERR_SHAPE
    assert L.iptq_metric_softmax(s.data_ptr(), p.data_ptr(), 4, 8, 0.0, 8, sc.sums.data_ptr(), sc.work.data_ptr(), None) == api.ERR_SCALE_RANGE
    assert L.iptq_metric_softmax(s.data_ptr(), p.data_ptr(), 4, 8, 3e-4, 9, sc.sums.data_ptr(), sc.work.data_ptr(), None) == api.ERR_BITS
    assert L.iptq_metric_gelu(None, None, 5, 1e-3, 0.03, 0, sc.sums.data_ptr(), sc.work.data_ptr(), None) == api.ERR_NULL
    assert L.iptq_metric_layernorm(s.data_ptr(), s.data_ptr(), 4, 6, g.data_ptr(), g.data_ptr(), None, 0.03, 0,
                                   sc.sums.data_ptr(), sc.work.data_ptr(), None) == api.ERR_SHAPE
    torch.cuda.synchronize()


def _oracle_analysis(orc, metric, layers, c_unit):
    """The same stage 1 / stage 2 with the oracle only."""
    out = []
    for name, kind, d in layers:
        cands = []
        if kind == "softmax":
            s, S = d["scores"], d["in_scale"]
            X = metric.softmax_float(s, S)
            for v in (0, 1, 2, 3):
                p = orc.softmax(s, orc.softmax_prepare(S, s.shape[1], 4 if v == 3 else 8, v))
                cands.append((v,) + metric.evaluate(X, metric.log2_deq(p) if v == 3 else metric.softmax_deq(p, 8),
                                                    metric.op_count(metric.SOFTMAX, v, s.shape[0], s.shape[1]), c_unit))
        elif kind == "gelu":
            x, S = d["x"], d["in_scale"]
            X = metric.gelu_float(x, S)
            for v in (0, 1, 2):
                try:
                    c = orc.gelu_prepare(S, d["in_bits"], d["out_scale"], d["out_zp"], 8, v)
                except orc.OracleError:
                    continue
                y = orc.gelu(x, c)
                cands.append((v,) + metric.evaluate(X, metric.affine_deq(y, d["out_scale"], d["out_zp"]),
                                                    metric.op_count(metric.GELU, v, x.size, 1), c_unit))
        else:
            x = d["x"]
            for v in (0, 1, 2):
                ptf = d["ptf"] if v == 2 else None
                gq, bq, c = orc.layernorm_prepare(d["gamma"], d["beta"], d["out_scale"], d["out_zp"], 8, v)
                y = orc.layernorm(x, gq, bq, c, ptf)
                X = metric.layernorm_float(x, d["gamma"], d["beta"], ptf)
                cands.append((v,) + metric.evaluate(X, metric.affine_deq(y, d["out_scale"], d["out_zp"]),
                                                    metric.op_count(metric.LAYERNORM, v, x.shape[0], x.shape[1]), c_unit))
        out.append((name, cands))
    return out


@pytest.mark.parametrize("c_unit", [1.0e6, 1.0e9])
def test_assignment_matches_oracle(api, orc, metric, c_unit):
    """DeiT-Tiny-sized encoder, two blocks, one image: 9 layers, up to 29 evaluations."""
    from paper_2511_15369_b200 import assign
    layers = list(synth.calibration_layers(192, 3, 197, 768, 2, 1, seed=4))
    an = assign.Analyzer(c_unit=c_unit)
    for name, kind, d in layers:
        if kind == "softmax":
            an.softmax_layer(name, _cu(d["scores"]), d["in_scale"])
        elif kind == "gelu":
            an.gelu_layer(name, _cu(d["x"]), d["in_scale"], d["in_bits"], d["out_scale"], d["out_zp"])
        else:
            an.layernorm_layer(name, _cu(d["x"]), d["gamma"], d["beta"], d["out_scale"], d["out_zp"],
                               ptf_shift=_cu(d["ptf"]))
    got, omega = an.finish()
    want = _oracle_analysis(orc, metric, layers, c_unit)
    assert len(got) == len(want) == 9
    omega_want = 0.0
    for g, (name, cands) in zip(got, want):
        assert g.name == name and [c.variant for c in g.candidates] == [c[0] for c in cands]
        for gc, (v, q, p, t) in zip(g.candidates, cands):
            assert abs(gc.sqnr_db - q) <= 1e-7 and abs(gc.perturbation - p) <= REL * p and abs(gc.term - t) <= 1e-9 * t
        terms = [c[3] for c in cands]
        best = metric.select(terms)
        omega_want += terms[best]
        runner_up = max([t for i, t in enumerate(terms) if i != best], default=-math.inf)
        if terms[best] - runner_up > 1e-8 * terms[best]:       # a clear winner must be the same on both sides
            assert g.choice == cands[best][0], (name, terms)
    assert abs(omega - omega_want) <= 1e-8 * omega_want
    tables = assign.block_tables(got, 2)
    assert len(tables) == 2 and all(len(t) == 4 for t in tables)
