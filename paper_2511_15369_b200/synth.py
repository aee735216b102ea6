"""Seeded synthetic inputs shaped like the paper's DeiT / ViT / Swin workloads.

This module holds NONE of the method's integer arithmetic: it draws float
tensors with numpy, quantises them with the plain uniform quantiser of the
paper's background section (round(x / s) + z, clipped), and runs an fp64
"shadow" forward pass only to pick the scale of every intermediate tensor
(the job PTQ calibration does on real images).  Both the CUDA library and the
CPU oracle are fed from here; each side then derives its own integer constants
with its own ``*_prepare`` functions.

The inputs stand in for ImageNet / COCO activations and trained weights, which
are not available: logits ~ N(0, 3^2) with 1 % of each row set to +12, GELU
inputs ~ N(-0.3, 1.2^2) with a 0.5 % Laplace(0, 4) tail, LayerNorm inputs
~ N(0, 1) with 2 % of the channels scaled by 20, weights ~ N(0, 0.02^2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# ------------------------------------------------------------------ shapes


@dataclass(frozen=True)
class BlockShape:
    name: str
    B: int        # images (or windows, for Swin)
    N: int        # tokens per attention problem
    D: int        # embedding dim
    H: int        # heads
    dh: int       # head dim
    Dh: int       # MLP hidden dim
    has_bias: bool = False   # relative-position bias [H, N, N]

    @property
    def T(self) -> int:
        return self.B * self.N

    def gemm_ops(self) -> int:
        """2 * sum(M*N*K) of the real (unpadded) contractions of one block."""
        T, D, Dh, N, dh = self.T, self.D, self.Dh, self.N, self.dh
        lin = T * D * (3 * D) + T * D * D + 2 * T * D * Dh
        att = 2 * self.B * self.H * N * N * dh
        return 2 * (lin + att)


CONFIGS = {
    "cfg0": BlockShape("DeiT-Tiny b1", 1, 197, 192, 3, 64, 768),
    "cfg1": BlockShape("DeiT-Small b64", 64, 197, 384, 6, 64, 1536),
    "cfg2": BlockShape("ViT-Base b128", 128, 197, 768, 12, 64, 3072),
    "cfg3": BlockShape("Swin-Tiny stage1 b64", 64 * 64, 49, 96, 3, 32, 384, True),
}

# Swin-Tiny backbone at detection resolution (config 4): token grid 200 x 304.
SWIN_T_STAGES = [
    dict(dim=96, heads=3, depth=2, grid=(200, 304)),
    dict(dim=192, heads=6, depth=2, grid=(100, 152)),
    dict(dim=384, heads=12, depth=6, grid=(50, 76)),
    dict(dim=768, heads=24, depth=2, grid=(25, 38)),
]


def _rng(seed: int, stream: int) -> np.random.Generator:
    """Independent sub-stream ``stream`` of ``seed`` (fixed spawn order)."""
    return np.random.default_rng(np.random.SeedSequence(seed).spawn(stream + 1)[stream])


# ------------------------------------------------------------------ stand-alone non-linear inputs

def softmax_logits(rows: int, n: int, seed: int = 0) -> np.ndarray:
    """fp64 logits [rows, n]: N(0, 3^2); ceil(1 % of n) random positions per row set to +12."""
    g = _rng(seed, 0)
    x = g.normal(0.0, 3.0, size=(rows, n))
    k = max(1, math.ceil(0.01 * n))
    pos = np.argsort(g.random((rows, n)), axis=1)[:, :k]
    np.put_along_axis(x, pos, 12.0, axis=1)
    return x


def quantize_scores(logits: np.ndarray, scale: float) -> np.ndarray:
    return np.round(logits / scale).astype(np.int32)


SOFTMAX_SCALE_ACC = 3.0e-4          # accumulator-like scale: floor(1/S) = 3333
SOFTMAX_SCALE_8BIT = 12.0 / 127.0   # 8-bit-like scale: floor(1/S) = 10


def gelu_values(n: int, seed: int = 0) -> np.ndarray:
    """fp64 GELU inputs: N(-0.3, 1.2^2), 0.5 % replaced by Laplace(0, 4)."""
    g = _rng(seed, 1)
    x = g.normal(-0.3, 1.2, size=n)
    tail = g.random(n) < 0.005
    x[tail] = g.laplace(0.0, 4.0, size=int(tail.sum()))
    return x


def quantize_sym(x: np.ndarray, bits: int, dtype=np.int32):
    """Symmetric per-tensor quantiser: scale = max|x| / (2^(bits-1) - 1)."""
    qmax = (1 << (bits - 1)) - 1
    scale = float(np.abs(x).max()) / qmax
    q = np.clip(np.round(x / scale), -qmax - 1, qmax).astype(dtype)
    return q, scale


def ln_values(rows: int, dim: int, seed: int = 0):
    """fp64 LayerNorm inputs [rows, dim]: N(0,1) with a fixed random 2 % of channels x20,
    plus gamma ~ N(1, 0.1^2), beta ~ N(0, 0.1^2)."""
    g = _rng(seed, 2)
    x = g.normal(0.0, 1.0, size=(rows, dim))
    k = max(1, round(0.02 * dim))
    ch = g.choice(dim, size=k, replace=False)
    x[:, ch] *= 20.0
    gamma = g.normal(1.0, 0.1, size=dim).astype(np.float32)
    beta = g.normal(0.0, 0.1, size=dim).astype(np.float32)
    return x, gamma, beta, np.sort(ch)


def ptf_shifts(xq: np.ndarray) -> np.ndarray:
    """Per-channel power-of-two factors alpha_c in {0..3}: the channels are quantised
    at scale S * 2^alpha_c; pick alpha from each channel's range (host-side calibration)."""
    amax = np.abs(xq.astype(np.int64)).max(axis=0).astype(np.float64)
    ref = max(1.0, float(np.median(amax)))
    a = np.clip(np.floor(np.log2(np.maximum(amax, 1.0) / ref)), 0, 3)
    return a.astype(np.uint8)


def affine_out_quant(y: np.ndarray, bits: int = 8):
    """Asymmetric output quantiser from the range of an fp64 reference:
    scale = (max - min) / (2^bits - 1), zero point placed in the signed range."""
    lo, hi = float(y.min()), float(y.max())
    lo, hi = min(lo, 0.0), max(hi, 0.0)
    scale = (hi - lo) / ((1 << bits) - 1)
    zp = int(round(-lo / scale)) - (1 << (bits - 1))
    return scale, zp


def calibration_layers(D: int, H: int, N: int, Dh: int, depth: int, batch: int, seed: int = 0):
    """Seeded calibration activations for every non-linear layer of a ViT encoder, in execution order: per block
    LN1, Softmax, LN2, GELU, then the final LayerNorm (4 * depth + 1 layers; ViT-Base: 49).  Each layer draws from
    the distribution of its kind (``ln_values`` / ``softmax_logits`` / ``gelu_values``) with its own seed and is
    quantised the way the block generator does it.  Yields (name, kind, dict of host arrays and scales), one layer
    at a time so that only one layer's activations are alive."""
    def ln(name, k):
        xf, gamma, beta, _ = ln_values(batch * N, D, seed=seed * 1000 + k)
        xq, S = quantize_sym(xf, 8, np.int8)
        So, zp = affine_out_quant(layernorm_ref(xq[:256].astype(np.float64), gamma, beta))
        return name, "layernorm", dict(x=xq, in_scale=S, gamma=gamma, beta=beta, out_scale=So, out_zp=zp,
                                       ptf=ptf_shifts(xq))
    k = 0
    for i in range(depth):
        yield ln("blk%d.ln1" % i, k); k += 1
        s = quantize_scores(softmax_logits(batch * H * N, N, seed=seed * 1000 + k), SOFTMAX_SCALE_ACC); k += 1
        yield "blk%d.softmax" % i, "softmax", dict(scores=s, in_scale=SOFTMAX_SCALE_ACC)
        yield ln("blk%d.ln2" % i, k); k += 1
        xg, S = quantize_sym(gelu_values(batch * N * Dh, seed=seed * 1000 + k), 16); k += 1
        So, zp = affine_out_quant(gelu_ref(xg[:4096] * S))
        yield "blk%d.gelu" % i, "gelu", dict(x=xg, in_scale=S, in_bits=16, out_scale=So, out_zp=zp)
    yield ln("final.ln", k)


# ------------------------------------------------------------------ fp64 references (for calibration / error reports)

def gelu_ref(x):
    from math import erf
    v = np.vectorize(erf)
    return 0.5 * x * (1.0 + v(x / math.sqrt(2.0)))


def layernorm_ref(x, gamma, beta):
    mu = x.mean(axis=-1, keepdims=True)
    sd = x.std(axis=-1, keepdims=True)
    sd = np.where(sd == 0, 1.0, sd)
    return (x - mu) / sd * gamma + beta


def softmax_ref(x):
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


# ------------------------------------------------------------------ weights

def quantize_weight(w: np.ndarray, bits: int = 8):
    """Symmetric per-output-channel weight quantiser.  Returns (int8 values, scales[N])."""
    qmax = (1 << (bits - 1)) - 1
    s = np.abs(w).max(axis=1) / qmax
    s = np.where(s == 0, 1.0, s)
    q = np.clip(np.round(w / s[:, None]), -qmax - 1, qmax).astype(np.int8)
    return q, s


def pack_int4(q: np.ndarray) -> np.ndarray:
    """Pack int4 values [N, K] two per byte: element k in byte k//2, even k in the low nibble."""
    assert q.shape[1] % 2 == 0
    u = (q.astype(np.int16) & 15).astype(np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


# ------------------------------------------------------------------ encoder block

@dataclass
class LinearSpec:
    w: np.ndarray            # int8 [N, K] (unpacked values, also for 4-bit)
    w_packed: np.ndarray     # what the library is given: int8 [N,K] or uint8 [N,K/2]
    bias: np.ndarray         # int32 [N], input zero-point already folded in
    ratio: np.ndarray        # fp64 [N]: S_x * S_w[n] / S_out
    out_zp: int = 0
    res_ratio: float | None = None   # S_res / S_out of the residual branch (before the 2^-16 widening)
    res_zp: int = 0


@dataclass
class BlockSpec:
    shape: BlockShape
    w_bits: int
    x: np.ndarray                                  # int8 [T, D]
    ln1: dict = field(default_factory=dict)        # gamma, beta (float32), out_scale, out_zp
    ln2: dict = field(default_factory=dict)
    qkv: LinearSpec | None = None
    proj: LinearSpec | None = None
    fc1: LinearSpec | None = None                  # ratio = S_x*S_w[n] / S_gelu_in
    fc2: LinearSpec | None = None
    softmax_scale: float = 0.0                     # scale of the int32 scores (1/sqrt(dh) folded in)
    pv_ratio: float = 0.0                          # 2^-(a_bits-1) * S_v / S_attn
    gelu: dict = field(default_factory=dict)       # in_scale, in_bits, out_scale, out_zp
    attn_bias: np.ndarray | None = None            # int32 [H, N, N] at the score scale
    mask_id: np.ndarray | None = None              # uint8 [B, N]
    a_bits: int = 8                                # activation width (8, or 6 for W6A6)


def make_block(shape: BlockShape, seed: int = 0, w_bits: int = 8, gelu_in_bits: int = 16,
               calib_images: int = 2, mask_id: np.ndarray | None = None, a_bits: int = 8) -> BlockSpec:
    """Draw one encoder block (weights, input) and calibrate every intermediate scale
    with an fp64 shadow forward over the first ``calib_images`` attention problems.
    ``w_bits`` 8 / 6 / 4 and ``a_bits`` 8 / 6 give the W8A8, W6A6 and W4A8 settings (6-bit values are stored as
    int8, 4-bit weights are packed)."""
    qa = float((1 << (a_bits - 1)) - 1)             # largest activation code
    g = _rng(seed, 3)
    T, D, H, dh, Dh, N = shape.T, shape.D, shape.H, shape.dh, shape.Dh, shape.N
    # block input: the LayerNorm-input distribution
    xin, g1, b1, _ = ln_values(T, D, seed)
    x, Sx = quantize_sym(xin, a_bits, np.int8)
    del xin
    Tc = min(T, calib_images * N)
    Bc = Tc // N
    xc = x[:Tc].astype(np.float64) * Sx

    def draw_w(n, k, gain=1.0):
        return g.normal(0.0, 0.02, size=(n, k)) * gain, g.normal(0.0, 0.02, size=n) * gain

    def qlin(wf, bf, S_in, w_bits_):
        wq, Sw = quantize_weight(wf, w_bits_)
        bq = np.round(bf / (S_in * Sw)).astype(np.int32)
        wp = pack_int4(wq) if w_bits_ == 4 else wq
        return wq, Sw, bq, wp

    spec = BlockSpec(shape=shape, w_bits=w_bits, x=x, a_bits=a_bits)
    # ---- LN1
    h1 = layernorm_ref(xc, g1, b1)
    S_h1 = float(np.abs(h1).max()) / qa
    # the block's activations carry one scale per tensor, so the power-of-two factors LN_PTF takes are all 2^0
    spec.ln1 = dict(gamma=g1, beta=b1, out_scale=S_h1, out_zp=0, ptf=np.zeros(shape.D, np.uint8))
    h1 = np.clip(np.round(h1 / S_h1), -qa - 1, qa) * S_h1
    # ---- QKV; a gain on the q/k rows puts the logits on config 0's N(0, 3^2) spread
    wf, bf = draw_w(3 * D, D)
    q0 = h1 @ wf[:D].T + bf[:D]
    k0 = h1 @ wf[D:2 * D].T + bf[D:2 * D]
    lg = np.einsum("bnhd,bmhd->bhnm", q0.reshape(Bc, N, H, dh), k0.reshape(Bc, N, H, dh)) / math.sqrt(dh)
    gain = math.sqrt(3.0 / float(lg.std()))
    wf[:2 * D] *= gain
    bf[:2 * D] *= gain
    wq, Sw, bq, wp = qlin(wf, bf, S_h1, w_bits)
    qkv = h1 @ (wq * Sw[:, None]).T + bq * (S_h1 * Sw)
    S_qkv = float(np.abs(qkv).max()) / qa
    spec.qkv = LinearSpec(wq, wp, bq, S_h1 * Sw / S_qkv)
    qkv = np.clip(np.round(qkv / S_qkv), -qa - 1, qa) * S_qkv
    # ---- attention
    spec.softmax_scale = S_qkv * S_qkv / math.sqrt(dh)
    qh = qkv[:, :D].reshape(Bc, N, H, dh)
    kh = qkv[:, D:2 * D].reshape(Bc, N, H, dh)
    vh = qkv[:, 2 * D:].reshape(Bc, N, H, dh)
    lg = np.einsum("bnhd,bmhd->bhnm", qh, kh) / math.sqrt(dh)
    if shape.has_bias:
        bias_f = g.normal(0.0, 1.0, size=(H, N, N))
        spec.attn_bias = np.round(bias_f / spec.softmax_scale).astype(np.int32)
        lg = lg + spec.attn_bias[None] * spec.softmax_scale
    if mask_id is not None:
        spec.mask_id = np.ascontiguousarray(mask_id, dtype=np.uint8)
        mm = spec.mask_id[:Bc, :, None] != spec.mask_id[:Bc, None, :]
        lg = np.where(mm[:, None], -1e9, lg)
    P = softmax_ref(lg)
    att = np.einsum("bhnm,bmhd->bnhd", P, vh).reshape(Tc, D)
    # floor on the scale: the dyadic requantiser takes ratios below 1/4
    S_att = max(float(np.abs(att).max()) / qa, 4.2 * (2.0 ** -(a_bits - 1)) * S_qkv)
    spec.pv_ratio = (2.0 ** -(a_bits - 1)) * S_qkv / S_att
    att = np.clip(np.round(att / S_att), -qa - 1, qa) * S_att
    # ---- proj + residual
    wf, bf = draw_w(D, D)
    wq, Sw, bq, wp = qlin(wf, bf, S_att, w_bits)
    x1 = att @ (wq * Sw[:, None]).T + bq * (S_att * Sw) + xc
    S_x1 = float(np.abs(x1).max()) / qa
    spec.proj = LinearSpec(wq, wp, bq, S_att * Sw / S_x1, 0, Sx / S_x1, 0)
    x1 = np.clip(np.round(x1 / S_x1), -qa - 1, qa) * S_x1
    # ---- LN2
    g2 = g.normal(1.0, 0.1, size=D).astype(np.float32)
    b2 = g.normal(0.0, 0.1, size=D).astype(np.float32)
    h2 = layernorm_ref(x1, g2, b2)
    S_h2 = float(np.abs(h2).max()) / qa
    spec.ln2 = dict(gamma=g2, beta=b2, out_scale=S_h2, out_zp=0, ptf=np.zeros(shape.D, np.uint8))
    h2 = np.clip(np.round(h2 / S_h2), -qa - 1, qa) * S_h2
    # ---- FC1 + GELU; a gain puts the GELU input on config 0's N(-0.3, 1.2^2) spread
    wf, bf = draw_w(Dh, D)
    a0 = h2 @ wf.T + bf
    gain = 1.2 / float(a0.std())
    wf *= gain
    bf = bf * gain - 0.3
    wq, Sw, bq, wp = qlin(wf, bf, S_h2, w_bits)
    a = h2 @ (wq * Sw[:, None]).T + bq * (S_h2 * Sw)
    # widest GELU input (<= gelu_in_bits) whose per-channel requant ratio stays below 1/4
    while True:
        qmax_in = (1 << (gelu_in_bits - 1)) - 1
        S_gin = float(np.abs(a).max()) / qmax_in
        if gelu_in_bits == 8 or float((S_h2 * Sw / S_gin).max()) < 0.25:
            break
        gelu_in_bits -= 1
    spec.fc1 = LinearSpec(wq, wp, bq, S_h2 * Sw / S_gin)
    hid = gelu_ref(a)
    S_hid, zp_hid = affine_out_quant(hid, a_bits)
    spec.gelu = dict(in_scale=S_gin, in_bits=gelu_in_bits, out_scale=S_hid, out_zp=zp_hid)
    hid_q = np.clip(np.round(hid / S_hid) + zp_hid, -qa - 1, qa)
    hid = (hid_q - zp_hid) * S_hid
    # ---- FC2 + residual; the hidden zero point is folded into the bias
    wf, bf = draw_w(D, Dh)
    wq, Sw, bq, wp = qlin(wf, bf, S_hid, w_bits)
    bq = (bq.astype(np.int64) - zp_hid * wq.astype(np.int64).sum(axis=1)).astype(np.int32)
    yf = hid_q @ (wq * Sw[:, None]).T * S_hid + bq * (S_hid * Sw) + x1
    S_y = float(np.abs(yf).max()) / qa
    spec.fc2 = LinearSpec(wq, wp, bq, S_hid * Sw / S_y, 0, S_x1 / S_y, 0)
    return spec


# ------------------------------------------------------------------ Swin shifted-window labels

def swin_mask_ids(window: int = 7, shift: int = 3) -> np.ndarray:
    """Region label of every token of the last window in each direction after a cyclic shift:
    tokens with different labels must not attend to each other.  Returns the 4 label
    patterns [4, window*window] (interior, right edge, bottom edge, corner)."""
    def lab(n_edge):
        a = np.zeros(window, dtype=np.uint8)
        if n_edge:
            a[window - shift:] = 1
        return a
    out = []
    for eh in (0, 1):
        for ew in (0, 1):
            out.append((lab(eh)[:, None] * 2 + lab(ew)[None, :]).reshape(-1))
    return np.stack(out).astype(np.uint8)


# ------------------------------------------------------------------ Swin backbone layout (config 4)
# The tables below are pure index arithmetic (which token goes where); both the CUDA library and the oracle-side
# composition in the tests consume them.  Conventions (the paper describes none of this): the token grid is padded
# at the bottom/right to multiples of the window; shifted blocks roll the padded grid by -shift before the
# partition and back afterwards; tokens of one window attend to each other only if they carry the same label --
# the 3 x 3 region labels of the rolled grid for shifted blocks, 0 otherwise; padding tokens are zero rows that
# carry label 255, so no real token ever attends to them.

PAD_LABEL = 255


def swin_window_tables(B: int, Hh: int, Ww: int, shift: int, window: int = 7):
    """Returns (fwd, mask_id, rev, n_windows):
    fwd     int32 [B*nW*window^2]  source token row of every window-layout row (-1 = padding),
    mask_id uint8 [B*nW, window^2] attention labels,
    rev     int32 [B*Hh*Ww]        window-layout row holding every token's result."""
    Hp = -(-Hh // window) * window
    Wp = -(-Ww // window) * window
    nh, nw = Hp // window, Wp // window
    ii, jj = np.meshgrid(np.arange(Hp), np.arange(Wp), indexing="ij")      # positions in the rolled, padded grid
    si, sj = (ii + shift) % Hp, (jj + shift) % Wp                          # where each of them comes from
    real = (si < Hh) & (sj < Ww)
    src = np.where(real, si * Ww + sj, -1)

    def region(n, size):
        r = np.zeros(n, dtype=np.int64)
        if shift:
            r[size - window:size - shift] = 1
            r[size - shift:] = 2
        return r
    label = region(Hp, Hp)[:, None] * 3 + region(Wp, Wp)[None, :]
    label = np.where(real, label, PAD_LABEL)

    def to_windows(a):
        return a.reshape(nh, window, nw, window).transpose(0, 2, 1, 3).reshape(nh * nw, window * window)
    src_w, lab_w = to_windows(src), to_windows(label)
    nW = nh * nw
    fwd = np.empty((B, nW, window * window), dtype=np.int32)
    for b in range(B):
        fwd[b] = np.where(src_w >= 0, src_w + b * Hh * Ww, -1)
    mask_id = np.broadcast_to(lab_w.astype(np.uint8), (B, nW, window * window)).reshape(B * nW, window * window)
    rev = np.full(B * Hh * Ww, -1, dtype=np.int32)
    flat = fwd.reshape(-1)
    rows = np.nonzero(flat >= 0)[0]
    rev[flat[rows]] = rows.astype(np.int32)
    assert (rev >= 0).all()
    return fwd.reshape(-1), mask_id.copy(), rev, nW


def swin_merge_table(B: int, Hh: int, Ww: int) -> np.ndarray:
    """int32 [B*(Hh/2)*(Ww/2), 4]: the four tokens (even/even, odd/even, even/odd, odd/odd rows/columns of a
    2 x 2 patch) whose channels are concatenated by the patch merge; -1 where an odd grid has no token."""
    H2, W2 = -(-Hh // 2), -(-Ww // 2)
    i2, j2 = np.meshgrid(np.arange(H2), np.arange(W2), indexing="ij")
    out = np.empty((B, H2 * W2, 4), dtype=np.int32)
    for p, (di, dj) in enumerate(((0, 0), (1, 0), (0, 1), (1, 1))):
        i, j = 2 * i2 + di, 2 * j2 + dj
        ok = (i < Hh) & (j < Ww)
        t = np.where(ok, i * Ww + j, -1).reshape(-1)
        for b in range(B):
            out[b, :, p] = np.where(t >= 0, t + b * Hh * Ww, -1)
    return out.reshape(-1, 4)


@dataclass
class MergeSpec:
    gamma: np.ndarray       # float32 [4C]
    beta: np.ndarray        # float32 [4C]
    ln_out_scale: float
    w: np.ndarray           # int8 [2C, 4C]
    ratio: np.ndarray       # fp64 [2C]


def make_merge(C: int, seed: int) -> MergeSpec:
    """Patch-merge layer 4C -> 2C: LayerNorm(4C) then a bias-free linear, scales from an fp64 shadow pass."""
    g = _rng(seed, 4)
    xin, _, _, _ = ln_values(256, 4 * C, seed)
    xq, _ = quantize_sym(xin, 8, np.int8)
    gamma = g.normal(1.0, 0.1, size=4 * C).astype(np.float32)
    beta = g.normal(0.0, 0.1, size=4 * C).astype(np.float32)
    h = layernorm_ref(xq.astype(np.float64), gamma, beta)
    S_h = float(np.abs(h).max()) / 127.0
    h = np.clip(np.round(h / S_h), -128, 127) * S_h
    wf = g.normal(0.0, 0.02, size=(2 * C, 4 * C))
    wq, Sw = quantize_weight(wf, 8)
    o = h @ (wq * Sw[:, None]).T
    S_o = float(np.abs(o).max()) / 127.0
    return MergeSpec(gamma, beta, S_h, wq, S_h * Sw / S_o)


@dataclass
class SwinSpec:
    B: int
    stages: list            # per stage: dict(dim, heads, grid, blocks=[(BlockSpec, shift, fwd, rev, n_rows)], merge=(MergeSpec, table) or None)
    x: np.ndarray           # int8 [B*H0*W0, C0]


def make_swin(B: int = 2, stages=None, seed: int = 0, window: int = 7) -> SwinSpec:
    """Swin-Tiny-shaped backbone on a B x grid token field: per stage `depth` blocks (odd ones shifted by
    window // 2) followed, except after the last stage, by a patch merge.  Every block draws its own weights and
    calibrates its scales on its own synthetic input (see make_block)."""
    stages = SWIN_T_STAGES if stages is None else stages
    out = []
    for si, st in enumerate(stages):
        Hh, Ww = st["grid"]
        C, H = st["dim"], st["heads"]
        blocks = []
        for d in range(st["depth"]):
            shift = (window // 2) if d % 2 else 0
            fwd, mask_id, rev, nW = swin_window_tables(B, Hh, Ww, shift, window)
            shape = BlockShape("swin s%d b%d" % (si, d), B * nW, window * window, C, H, C // H, 4 * C, True)
            spec = make_block(shape, seed=seed + 100 * si + d, mask_id=mask_id, calib_images=4)
            spec.x = None                                   # the block's input comes from the layer before it
            blocks.append((spec, shift, fwd, rev))
        merge = None
        if si + 1 < len(stages):
            merge = (make_merge(C, seed + 100 * si + 50), swin_merge_table(B, Hh, Ww))
        out.append(dict(dim=C, heads=H, grid=(Hh, Ww), blocks=blocks, merge=merge))
    Hh, Ww = stages[0]["grid"]
    xin, _, _, _ = ln_values(B * Hh * Ww, stages[0]["dim"], seed)
    x, _ = quantize_sym(xin, 8, np.int8)
    return SwinSpec(B, out, x)


# ------------------------------------------------------------------ whole ViT / DeiT models (Sec. 4, latency table)

VIT_MODELS = {
    "DeiT-T": dict(D=192, H=3, depth=12),
    "DeiT-S": dict(D=384, H=6, depth=12),
    "DeiT-B": dict(D=768, H=12, depth=12),
}


@dataclass
class VitSpec:
    name: str
    B: int
    D: int
    H: int
    depth: int
    img_size: int
    patch: int
    classes: int
    image: np.ndarray           # int8 [B, 3, img, img]
    embed: LinearSpec           # patch rows [B*P, 3*patch*patch] -> [B*P, D]; residual = position rows
    pos: np.ndarray             # int8 [P, D] position embedding of the patch tokens (residual branch)
    cls_row: np.ndarray         # int8 [D]: class token + its position embedding, at the token scale
    blocks: list                # BlockSpec per encoder block (x = None: the input comes from the layer before)
    final_ln: dict              # gamma, beta, out_scale, out_zp
    head: LinearSpec            # [B, D] -> [B, classes]

    @property
    def N(self) -> int:
        return (self.img_size // self.patch) ** 2 + 1

    def gemm_ops(self) -> int:
        P = self.N - 1
        ops = 2 * self.B * P * self.D * 3 * self.patch * self.patch + 2 * self.B * self.D * self.classes
        return ops + sum(b.shape.gemm_ops() for b in self.blocks)


def make_vit(name: str = "DeiT-S", B: int = 8, seed: int = 0, img_size: int = 224, patch: int = 16,
             classes: int = 1000, depth: int | None = None) -> VitSpec:
    """A ViT/DeiT-shaped integer model with seeded random weights: patch embedding (+ position embedding through
    the residual branch of the linear layer), class token, `depth` encoder blocks, final LayerNorm, classifier.
    The front end is calibrated by an fp64 shadow pass over the first two images; every block calibrates on its own
    synthetic input (see make_block); the final LayerNorm and the classifier use fixed ranges (8 standard deviations
    and 6 standard deviations of a unit-variance input)."""
    m = VIT_MODELS[name]
    D, H = m["D"], m["H"]
    depth = m["depth"] if depth is None else depth
    g = _rng(seed, 5)
    gsz = img_size // patch
    P, K = gsz * gsz, 3 * patch * patch
    img_f = g.normal(0.0, 1.0, size=(B, 3, img_size, img_size))
    image, S_img = quantize_sym(img_f, 8, np.int8)
    del img_f
    # ---- patch embedding + position embedding (fp64 shadow on two images)
    Bc = min(B, 2)
    rows = image[:Bc].reshape(Bc, 3, gsz, patch, gsz, patch).transpose(0, 2, 4, 1, 3, 5).reshape(Bc * P, K)
    wf = g.normal(0.0, 0.02, size=(D, K))
    bf = g.normal(0.0, 0.02, size=D)
    wq, Sw = quantize_weight(wf, 8)
    bq = np.round(bf / (S_img * Sw)).astype(np.int32)
    pos_f = g.normal(0.0, 0.02, size=(P + 1, D))
    cls_f = g.normal(0.0, 0.02, size=D)
    pos, S_pos = quantize_sym(pos_f[1:], 8, np.int8)
    tok = rows.astype(np.float64) @ (wq * Sw[:, None]).T * S_img + bq * (S_img * Sw) + np.tile(pos * S_pos, (Bc, 1))
    S_tok = float(np.abs(tok).max()) / 127.0
    embed = LinearSpec(wq, wq, bq, S_img * Sw / S_tok, 0, S_pos / S_tok, 0)
    cls_row = np.clip(np.round((cls_f + pos_f[0]) / S_tok), -128, 127).astype(np.int8)
    # ---- encoder blocks
    shape = BlockShape("%s b%d" % (name, B), B, P + 1, D, H, D // H, 4 * D)
    blocks = []
    for i in range(depth):
        spec = make_block(shape, seed=seed + 1 + i, calib_images=2)
        spec.x = None
        blocks.append(spec)
    # ---- final LayerNorm and classifier
    gamma = g.normal(1.0, 0.1, size=D).astype(np.float32)
    beta = g.normal(0.0, 0.1, size=D).astype(np.float32)
    S_ln = 8.0 * float(np.abs(gamma).max()) / 127.0
    wf = g.normal(0.0, 0.02, size=(classes, D))
    bf = g.normal(0.0, 0.02, size=classes)
    wq, Sw = quantize_weight(wf, 8)
    bq = np.round(bf / (S_ln * Sw)).astype(np.int32)
    S_out = 6.0 * 0.02 * math.sqrt(D) / 127.0
    head = LinearSpec(wq, wq, bq, S_ln * Sw / S_out)
    return VitSpec(name, B, D, H, depth, img_size, patch, classes, image, embed, pos, cls_row, blocks,
                   dict(gamma=gamma, beta=beta, out_scale=S_ln, out_zp=0), head)
