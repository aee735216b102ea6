"""Oracle-side compositions: one encoder block and a whole ViT / DeiT forward pass from a parameter spec (any
object with the fields of ``synth.BlockSpec`` / ``synth.VitSpec``), using only the oracle's own functions and numpy
data movement.  TEST INFRASTRUCTURE ONLY, like the rest of this package."""
from __future__ import annotations

import numpy as np

import oracle


def _channel_requant(ratio):
    rq = [oracle.requant_prepare(float(r)) for r in ratio]
    return np.array([r.mult for r in rq], np.int32), np.array([r.shift for r in rq], np.int8)


def block_params(spec, table) -> dict:
    """Field dictionary of ``oracle.encoder_block`` for a block spec and a (softmax, gelu, ln1, ln2) variant table."""
    sm_v, gelu_v, ln1_v, ln2_v = table
    sh = spec.shape
    ab = getattr(spec, "a_bits", 8)                # activation width: 8, or 6 for the W6A6 setting
    d = dict(B=sh.B, N=sh.N, D=sh.D, H=sh.H, dh=sh.dh, Dh=sh.Dh, w_bits=4 if spec.w_bits == 4 else 8, act_bits=ab,
             sm_variant=sm_v, gelu_variant=gelu_v, ln1_variant=ln1_v, ln2_variant=ln2_v)
    for name, ln, var in (("ln1", spec.ln1, ln1_v), ("ln2", spec.ln2, ln2_v)):
        gq, bq, c = oracle.layernorm_prepare(ln["gamma"], ln["beta"], ln["out_scale"], ln["out_zp"], ab, var)
        d[name + "_gamma"], d[name + "_beta"], d[name], d[name + "_ptf"] = gq, bq, c, ln.get("ptf")
    for name, ls in (("qkv", spec.qkv), ("proj", spec.proj), ("fc1", spec.fc1), ("fc2", spec.fc2)):
        d["w_" + name], d["b_" + name] = ls.w_packed, ls.bias
        d["m_" + name], d["s_" + name] = _channel_requant(ls.ratio)
    # the logarithm candidate writes 4-bit codes and its P V product is at scale 2^-15 instead of 2^-7
    log2 = sm_v == oracle.SM_LOG2
    qa = 1 << (ab - 1)
    d["sm"] = oracle.softmax_prepare(spec.softmax_scale, sh.N, 4 if log2 else ab, sm_v)
    d["pv_rq"] = oracle.requant_prepare(spec.pv_ratio * qa / 32768 if log2 else spec.pv_ratio, 0, -qa, qa - 1)
    d["attn_bias"], d["mask_id"] = spec.attn_bias, spec.mask_id
    d["res1_rq"] = oracle.requant_prepare(spec.proj.res_ratio / 65536, zp=spec.proj.res_zp)
    d["res2_rq"] = oracle.requant_prepare(spec.fc2.res_ratio / 65536, zp=spec.fc2.res_zp)
    gl = spec.gelu
    d["gelu"] = oracle.gelu_prepare(gl["in_scale"], gl["in_bits"], gl["out_scale"], gl["out_zp"], ab, gelu_v)
    d["proj_zp"], d["fc2_zp"] = spec.proj.out_zp, spec.fc2.out_zp
    return d


def patch_rows(image: np.ndarray, patch: int) -> np.ndarray:
    """[B, C, H, W] -> [B * (H/patch) * (W/patch), C * patch * patch], rows in (b, py, px) order, columns (c, dy, dx)."""
    B, C, H, W = image.shape
    gh, gw = H // patch, W // patch
    r = image.reshape(B, C, gh, patch, gw, patch).transpose(0, 2, 4, 1, 3, 5)
    return np.ascontiguousarray(r.reshape(B * gh * gw, C * patch * patch))


def vit_forward(spec, table=(0, 0, 0, 0), return_tokens: bool = False):
    """int8 logits [B, classes] of the integer ViT described by ``spec`` (see synth.make_vit)."""
    B, N, D = spec.B, spec.N, spec.D
    P = N - 1
    e = spec.embed
    m, s = _channel_requant(e.ratio)
    rows = patch_rows(spec.image, spec.patch)
    res_rq = oracle.requant_prepare(e.res_ratio / 65536, zp=e.res_zp)
    emb = oracle.linear(rows, e.w_packed, e.bias, m, s, e.out_zp, residual=np.ascontiguousarray(np.tile(spec.pos, (B, 1))),
                        residual_rq=res_rq)
    x = np.empty((B, N, D), dtype=np.int8)
    x[:, 0] = spec.cls_row
    x[:, 1:] = emb.reshape(B, P, D)
    x = np.ascontiguousarray(x.reshape(B * N, D))
    for b in spec.blocks:
        x = oracle.encoder_block(x, block_params(b, table))
    cls = np.ascontiguousarray(x.reshape(B, N, D)[:, 0])
    f = spec.final_ln
    gq, bq, c = oracle.layernorm_prepare(f["gamma"], f["beta"], f["out_scale"], f["out_zp"], 8, 0)
    h = oracle.layernorm(cls, gq, bq, c)
    hd = spec.head
    m, s = _channel_requant(hd.ratio)
    logits = oracle.linear(h, hd.w_packed, hd.bias, m, s, hd.out_zp)
    return (logits, x) if return_tokens else logits
