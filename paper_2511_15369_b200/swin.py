"""Swin-shaped backbone as a sequence of C-ABI calls: per block a row gather into 7x7 windows (cyclic shift and
padding folded into the gather table), the integer encoder block on the windows (relative-position bias, attention
labels), and the gather back; between stages the 2x2 patch merge (gather, integer LayerNorm, INT8 linear).
Host logic only: tables and parameters are prepared once, every step of the data path runs in the library."""
from __future__ import annotations

import numpy as np
import torch

from . import api


class SwinBackbone:
    def __init__(self, spec, table=(api.SM_BITEXP, api.GELU_POLY4, api.LN_SHIFT, api.LN_SHIFT), device="cuda"):
        self.spec = spec
        self.layers = []
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
        for st in spec.stages:
            C = st["dim"]
            for bspec, shift, fwd, rev in st["blocks"]:
                blk = api.EncoderBlock(bspec, table, device)
                n_rows = bspec.shape.T
                self.layers.append(("block", blk, dev(fwd.reshape(-1, 1)), dev(rev.reshape(-1, 1)),
                                    torch.empty((n_rows, C), dtype=torch.int8, device=device),
                                    torch.empty((n_rows, C), dtype=torch.int8, device=device)))
            if st["merge"] is not None:
                m, tab = st["merge"]
                gq, bq, lc = api.layernorm_prepare(m.gamma, m.beta, m.ln_out_scale, 0)
                mult, shift = api.channel_requant_prepare(m.ratio)
                ws = api.Workspace(api.linear_workspace_bytes(tab.shape[0], 2 * C, 4 * C))
                self.layers.append(("merge", dev(tab), dev(gq), dev(bq), lc, dev(m.w), dev(mult), dev(shift), ws))

    def __call__(self, x):
        for L in self.layers:
            if L[0] == "block":
                _, blk, fwd, rev, xw, yw = L
                api.gather_rows(x, fwd, out=xw)
                blk(xw, yw)
                x = api.gather_rows(yw, rev)
            else:
                _, tab, gq, bq, lc, w, mult, shift, ws = L
                g = api.gather_rows(x, tab)
                h = api.layernorm(g, gq, bq, lc)
                x = api.linear(h, w, None, mult, shift, ws)
        return x

    def check(self):
        for L in self.layers:
            (L[1].ws if L[0] == "block" else L[8]).check()

    def gemm_ops(self) -> int:
        ops = 0
        for st in self.spec.stages:
            for bspec, *_ in st["blocks"]:
                ops += bspec.shape.gemm_ops()
            if st["merge"] is not None:
                m, tab = st["merge"]
                ops += 2 * tab.shape[0] * m.w.shape[0] * m.w.shape[1]
        return ops
