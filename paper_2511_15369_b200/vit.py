"""Whole ViT / DeiT forward pass as a sequence of C-ABI calls (the models of the paper's latency table, Sec. 4.3):
patch rows -> INT8 patch embedding with the position embedding on the residual branch -> class token inserted by a
row gather -> `depth` integer encoder blocks -> class rows gathered -> integer LayerNorm -> INT8 classifier.
Host logic only: parameters and tables are prepared once, every step of the data path runs in the library; all
buffers are allocated up front so that a forward pass can be captured in a CUDA graph."""
from __future__ import annotations

import numpy as np
import torch

from . import api


class VitModel:
    def __init__(self, spec, table=(api.SM_BITEXP, api.GELU_POLY4, api.LN_SHIFT, api.LN_SHIFT), device="cuda"):
        self.spec = spec
        B, N, D = spec.B, spec.N, spec.D
        P = N - 1
        K = 3 * spec.patch * spec.patch
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
        i8 = lambda *shape: torch.empty(shape, dtype=torch.int8, device=device)
        # patch embedding; its output lands in the first B*P rows of tok_src, the class row sits behind them
        e = spec.embed
        m, s = api.channel_requant_prepare(e.ratio)
        self.embed = dict(w=dev(e.w_packed), b=dev(e.bias), m=dev(m), s=dev(s), zp=e.out_zp,
                          res=dev(np.tile(spec.pos, (B, 1))), res_rq=api.requant_prepare(e.res_ratio / 65536.0, zp=e.res_zp),
                          ws=api.Workspace(api.linear_workspace_bytes(B * P, D, K), device))
        self.patch_rows = i8(B * P, K)
        self.tok_src = i8(B * P + 1, D)
        self.tok_src[B * P].copy_(dev(spec.cls_row))
        idx = np.empty((B, N), dtype=np.int32)
        idx[:, 0] = B * P
        idx[:, 1:] = np.arange(B * P, dtype=np.int32).reshape(B, P)
        self.tok_index = dev(idx.reshape(-1, 1))
        self.cls_index = dev((np.arange(B, dtype=np.int32) * N).reshape(-1, 1))
        self.x = [i8(B * N, D), i8(B * N, D)]
        self.blocks = [api.EncoderBlock(b, table, device) for b in spec.blocks]
        # final LayerNorm on the class rows, classifier
        f = spec.final_ln
        gq, bq, self.ln_c = api.layernorm_prepare(f["gamma"], f["beta"], f["out_scale"], f["out_zp"])
        self.ln_g, self.ln_b = dev(gq), dev(bq)
        self.cls_in, self.cls_ln = i8(B, D), i8(B, D)
        # the linear kernel wants N % 16 == 0: the classifier is padded with zero rows whose outputs are dropped
        h = spec.head
        npad = (spec.classes + 15) // 16 * 16
        pad = npad - spec.classes
        m, s = api.channel_requant_prepare(np.concatenate([h.ratio, np.repeat(h.ratio[-1:], pad)]))
        w = np.concatenate([h.w_packed, np.zeros((pad, D), dtype=h.w_packed.dtype)])
        b = np.concatenate([h.bias, np.zeros(pad, dtype=h.bias.dtype)])
        self.head = dict(w=dev(w), b=dev(b), m=dev(m), s=dev(s), zp=h.out_zp,
                         ws=api.Workspace(api.linear_workspace_bytes(B, npad, D), device))
        self.logits_padded = i8(B, npad)
        self.logits = self.logits_padded[:, :spec.classes]

    def __call__(self, image):
        """image: device int8 [B, 3, img, img] -> int8 logits [B, classes] (a view of a buffer of the model)."""
        sp, e, h = self.spec, self.embed, self.head
        P = sp.N - 1
        api.patchify(image, sp.patch, out=self.patch_rows)
        api.linear(self.patch_rows, e["w"], e["b"], e["m"], e["s"], e["ws"], e["zp"], residual=e["res"],
                   residual_rq=e["res_rq"], out=self.tok_src[:sp.B * P])
        api.gather_rows(self.tok_src, self.tok_index, out=self.x[0])
        cur = 0
        for blk in self.blocks:
            blk(self.x[cur], self.x[cur ^ 1])
            cur ^= 1
        api.gather_rows(self.x[cur], self.cls_index, out=self.cls_in)
        api.layernorm(self.cls_in, self.ln_g, self.ln_b, self.ln_c, out=self.cls_ln)
        api.linear(self.cls_ln, h["w"], h["b"], h["m"], h["s"], h["ws"], h["zp"], out=self.logits_padded)
        return self.logits

    def check(self):
        self.embed["ws"].check()
        self.head["ws"].check()
        for blk in self.blocks:
            blk.ws.check()

    def launches_per_forward(self) -> int:
        return 3 + 7 * len(self.blocks) + 3
