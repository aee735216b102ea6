"""Stages 1 and 2 of the assignment pipeline (Sec. 3.5, pipeline figure): every non-linear layer is run with each
candidate approximation function on calibration activations, scored with the Unified Metric of Eqs. (16)-(20), and
given the candidate with the largest term.

All arithmetic runs in the library: the integer candidates are the deployed kernels (``iptq_softmax`` /
``iptq_gelu`` / ``iptq_layernorm``), the float layer and the error sums are the ``iptq_metric_*`` reductions, the
scoring is ``iptq_metric_term`` / ``iptq_metric_select``.  This module only sequences the calls and keeps the
results; it synchronises with the device once, in ``finish()``.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import api

SOFTMAX_CANDIDATES = (api.SM_BITEXP, api.SM_SHIFTMAX, api.SM_POLY, api.SM_LOG2)
GELU_CANDIDATES = (api.GELU_POLY4, api.GELU_POLY2, api.GELU_SHIFT)
LN_CANDIDATES = (api.LN_SHIFT, api.LN_NEWTON, api.LN_PTF)


@dataclass
class Candidate:
    variant: int
    op_count: float
    slot: int                      # row of the device sums buffer
    sum_x2: float = float("nan")
    sum_err2: float = float("nan")
    sqnr_db: float = float("nan")
    perturbation: float = float("nan")
    term: float = float("nan")


@dataclass
class Layer:
    name: str
    kind: int
    candidates: list = field(default_factory=list)
    choice: int = -1               # variant id of the selected candidate


class _Slot:
    """MetricScratch look-alike that points one evaluation at its own row of the sums buffer."""

    def __init__(self, work, sums_row):
        self.work = work
        self.sums = sums_row


class Analyzer:
    def __init__(self, device="cuda", max_evaluations=256, c_unit=1.0e6):
        self.device = device
        self.c_unit = float(c_unit)
        self.work = torch.empty(api.METRIC_WORK_BYTES // 8, dtype=torch.float64, device=device)
        self.sums = torch.zeros((max_evaluations, 2), dtype=torch.float64, device=device)
        self.layers: list[Layer] = []
        self.n_eval = 0
        self._keep = []            # tables referenced by raw pointers until finish()

    def _slot(self):
        if self.n_eval >= self.sums.shape[0]:
            raise RuntimeError("more evaluations than max_evaluations")
        s = _Slot(self.work, self.sums[self.n_eval])
        self.n_eval += 1
        return s

    def softmax_layer(self, name, scores, in_scale, variants=SOFTMAX_CANDIDATES, out_bits=8):
        """scores: device int32 [rows, n] at scale in_scale."""
        rows, n = scores.shape
        layer = Layer(name, api.LAYER_SOFTMAX)
        probs = torch.empty((rows, n), dtype=torch.uint8, device=scores.device)
        for v in variants:
            bits = 4 if v == api.SM_LOG2 else out_bits         # the logarithm candidate writes 4-bit codes
            try:
                c = api.softmax_prepare(in_scale, n, bits, v)
            except api.IptqError:
                continue                   # this candidate has no integer constants at this scale
            self._keep.append(api.softmax_table(c, scores.device))
            api.softmax(scores, c, out=probs)
            slot = self._slot()
            api.metric_softmax(scores, probs, in_scale, api.PROBS_LOG2 if v == api.SM_LOG2 else bits, scratch=slot)
            layer.candidates.append(Candidate(v, api.op_count(api.LAYER_SOFTMAX, v, rows, n), self.n_eval - 1))
        self.layers.append(layer)
        return layer

    def gelu_layer(self, name, x, in_scale, in_bits, out_scale, out_zp, variants=GELU_CANDIDATES, out_bits=8):
        """x: device int32 (any shape) at scale in_scale, in_bits wide."""
        layer = Layer(name, api.LAYER_GELU)
        y = torch.empty(x.shape, dtype=torch.int8, device=x.device)
        for v in variants:
            try:
                c = api.gelu_prepare(in_scale, in_bits, out_scale, out_zp, out_bits, v)
            except api.IptqError:
                continue                   # this candidate has no integer constants at this scale / width
            api.gelu(x, c, out=y)
            slot = self._slot()
            api.metric_gelu(x, y, in_scale, out_scale, out_zp, scratch=slot)
            layer.candidates.append(Candidate(v, api.op_count(api.LAYER_GELU, v, x.numel(), 1), self.n_eval - 1))
        self.layers.append(layer)
        return layer

    def layernorm_layer(self, name, x, gamma, beta, out_scale, out_zp, variants=LN_CANDIDATES, ptf_shift=None,
                        out_bits=8):
        """x: device int8 [rows, dim]; gamma, beta: host float32 [dim]; ptf_shift: device uint8 [dim], used by the
        LN_PTF candidate only (the other candidates read x as it is)."""
        rows, dim = x.shape
        layer = Layer(name, api.LAYER_LAYERNORM)
        g = torch.from_numpy(np.ascontiguousarray(gamma, dtype=np.float32)).to(x.device)
        b = torch.from_numpy(np.ascontiguousarray(beta, dtype=np.float32)).to(x.device)
        y = torch.empty((rows, dim), dtype=torch.int8, device=x.device)
        for v in variants:
            if v == api.LN_PTF and ptf_shift is None:
                continue
            gq, bq, c = api.layernorm_prepare(gamma, beta, out_scale, out_zp, out_bits, v)
            gqd, bqd = torch.from_numpy(gq).to(x.device), torch.from_numpy(bq).to(x.device)
            ptf = ptf_shift if v == api.LN_PTF else None
            api.layernorm(x, gqd, bqd, c, ptf, out=y)
            slot = self._slot()
            api.metric_layernorm(x, y, g, b, out_scale, out_zp, ptf, scratch=slot)
            layer.candidates.append(Candidate(v, api.op_count(api.LAYER_LAYERNORM, v, rows, dim), self.n_eval - 1))
        self.layers.append(layer)
        return layer

    def finish(self):
        """Reads the sums back (the only synchronisation), scores every candidate and selects per layer.
        Returns (layers, Omega) with Omega the sum of the selected terms, Eq. (16)."""
        host = self.sums[:max(self.n_eval, 1)].cpu().numpy()
        omega = 0.0
        for layer in self.layers:
            for cand in layer.candidates:
                cand.sum_x2, cand.sum_err2 = float(host[cand.slot, 0]), float(host[cand.slot, 1])
                cand.sqnr_db = api.sqnr_db(cand.sum_x2, cand.sum_err2)
                cand.perturbation = cand.sum_err2
                cand.term = api.metric_term(cand.sqnr_db, cand.perturbation, cand.op_count, self.c_unit)
            best = api.metric_select([c.term for c in layer.candidates])
            layer.choice = layer.candidates[best].variant
            omega += layer.candidates[best].term
        self._keep.clear()
        return self.layers, omega


def block_tables(layers, n_blocks):
    """Per-block (softmax, gelu, ln1, ln2) variant tuples from layers named 'blk{i}.{ln1|softmax|ln2|gelu}'."""
    by_name = {l.name: l.choice for l in layers}
    return [(by_name["blk%d.softmax" % i], by_name["blk%d.gelu" % i], by_name["blk%d.ln1" % i],
             by_name["blk%d.ln2" % i]) for i in range(n_blocks)]
