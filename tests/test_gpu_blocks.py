"""GPU parity of the tensor-core paths (INT8 GEMM carrier, fused MLP, fused attention, encoder block):
bit-exact against the CPU oracle on the same seeded inputs, through the C-ABI."""
import numpy as np
import pytest

from paper_2511_15369_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2511_15369_b200 import api as _api
    _api.lib()
    return _api


def _cu(a):
    import torch
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _mismatch(got, want):
    bad = np.argwhere(got != want)
    return "%d of %d differ; first at %s: got %s want %s" % (
        len(bad), got.size, bad[:3].tolist(), got[tuple(bad[0])] if len(bad) else None,
        want[tuple(bad[0])] if len(bad) else None)


def _linear_case(rng, M, N, K, w_bits=8):
    x = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    lim = 8 if w_bits == 4 else 128
    w = rng.integers(-lim, lim, size=(N, K)).astype(np.int8)
    bias = rng.integers(-3000, 3000, size=N).astype(np.int32)
    ratios = 2.0 ** rng.uniform(-12, -7, size=N) * (16 if w_bits == 4 else 1)
    return x, w, bias, ratios


# the last two shapes are long and large enough for CTA pairs: an odd number of channel tiles whose last one is ragged
# (2064 = 16 x 128 + 16), and a ragged last token tile with a reduction that ends inside a 128-byte block; the one
# before them is a long reduction over few tiles, which takes half-width tiles
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (197, 384, 384), (300, 1152, 384), (1000, 384, 1536),
                                   (77, 96, 96), (130, 288, 96), (256, 16, 16), (5, 144, 272),
                                   (2600, 384, 1536), (7100, 2064, 1536), (29000, 512, 1552)])
def test_linear_parity(api, orc, M, N, K):
    rng = np.random.default_rng(M + N + K)
    x, w, bias, ratios = _linear_case(rng, M, N, K)
    mo, so = [], []
    for r in ratios:
        q = orc.requant_prepare(r)
        mo.append(q.mult)
        so.append(q.shift)
    mo, so = np.array(mo, np.int32), np.array(so, np.int8)
    ma, sa = api.channel_requant_prepare(ratios)
    assert (ma == mo).all() and (sa == so).all()
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K))
    want = orc.linear(x, w, bias, mo, so, out_zp=3)
    got = api.linear(_cu(x), _cu(w), _cu(bias), _cu(ma), _cu(sa), ws, out_zp=3).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)
    # residual branch, no bias
    res = rng.integers(-128, 128, size=(M, N)).astype(np.int8)
    rro = orc.requant_prepare(0.9 / 65536, zp=-4)
    rra = api.requant_prepare(0.9 / 65536, zp=-4)
    want = orc.linear(x, w, None, mo, so, out_zp=-2, residual=res, residual_rq=rro)
    got = api.linear(_cu(x), _cu(w), None, _cu(ma), _cu(sa), ws, out_zp=-2, residual=_cu(res), residual_rq=rra).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)


@pytest.mark.parametrize("M,N,K", [(300, 160, 96), (2600, 384, 1536)])
def test_linear_large_shifts_and_biases(api, orc, M, N, K):
    """Channel groups whose shifts are all small, all large and mixed (the epilogue treats the zero point differently
    when every channel of a 32-channel group has a small shift), with biases that dwarf the sums."""
    rng = np.random.default_rng(M)
    x, w, _, _ = _linear_case(rng, M, N, K)
    ratios = 2.0 ** rng.uniform(-12, -7, size=N)
    ratios[32:64] = 2.0 ** rng.uniform(-27, -23, size=32)           # shifts of 23 .. 27 beyond the 32 of hi32
    ratios[64:96:3] = 2.0 ** rng.uniform(-26, -22, size=len(ratios[64:96:3]))
    bias = rng.integers(-3000, 3000, size=N).astype(np.int32)
    bias[32:96] = rng.integers(-(1 << 30), 1 << 30, size=64).astype(np.int32)
    bias[100] = (1 << 31) - 1 - (1 << 26)
    bias[101] = -(1 << 31) + (1 << 26)
    ma, sa = api.channel_requant_prepare(ratios)
    assert sa[32:64].min() >= 22 and sa[:32].max() <= 12
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K))
    for zp in (3, -128, 127):
        want = orc.linear(x, w, bias, ma, sa, out_zp=zp)
        got = api.linear(_cu(x), _cu(w), _cu(bias), _cu(ma), _cu(sa), ws, out_zp=zp).cpu().numpy()
        ws.check()
        assert (got == want).all(), _mismatch(got, want)
    assert len(np.unique(want[:, 32:96])) > 20


@pytest.mark.parametrize("out_bits", [6, 4])
def test_linear_narrow_outputs(api, orc, out_bits):
    """Outputs clamped to a signed range narrower than 8 bits (W6A6 activations), plain and residual epilogue."""
    M, N, K = 333, 384, 192
    rng = np.random.default_rng(out_bits)
    x, w, bias, ratios = _linear_case(rng, M, N, K)
    ma, sa = api.channel_requant_prepare(ratios)
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K))
    want = orc.linear(x, w, bias, ma, sa, out_zp=1, out_bits=out_bits)
    got = api.linear(_cu(x), _cu(w), _cu(bias), _cu(ma), _cu(sa), ws, out_zp=1, out_bits=out_bits).cpu().numpy()
    ws.check()
    q = 1 << (out_bits - 1)
    assert want.min() == -q and want.max() == q - 1
    assert (got == want).all(), _mismatch(got, want)
    res = rng.integers(-q, q, size=(M, N)).astype(np.int8)
    rro, rra = orc.requant_prepare(0.9 / 65536, zp=-1), api.requant_prepare(0.9 / 65536, zp=-1)
    want = orc.linear(x, w, None, ma, sa, out_zp=-2, residual=res, residual_rq=rro, out_bits=out_bits)
    got = api.linear(_cu(x), _cu(w), None, _cu(ma), _cu(sa), ws, out_zp=-2, residual=_cu(res), residual_rq=rra,
                     out_bits=out_bits).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)
    with pytest.raises(api.IptqError):
        api.linear(_cu(x), _cu(w), None, _cu(ma), _cu(sa), ws, out_bits=9)


def test_linear_w4(api, orc):
    rng = np.random.default_rng(44)
    M, N, K = 200, 256, 384
    x, w, bias, ratios = _linear_case(rng, M, N, K, 4)
    wp = synth.pack_int4(w)
    ma, sa = api.channel_requant_prepare(ratios)
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K, 4))
    want = orc.linear(x, wp, bias, ma, sa, w_bits=4)
    got = api.linear(_cu(x), _cu(wp), _cu(bias), _cu(ma), _cu(sa), ws, w_bits=4).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)
    assert (want == orc.linear(x, w, bias, ma, sa)).all()


def test_mlp_w4(api, orc):
    """FC1 + GELU + FC2 with packed 4-bit weights (both matrices unpacked by one launch), with and without FC2."""
    rng = np.random.default_rng(45)
    M, D, Dh = 150, 96, 384
    x = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    w1 = rng.integers(-8, 8, size=(Dh, D)).astype(np.int8)
    w2 = rng.integers(-8, 8, size=(D, Dh)).astype(np.int8)
    b1 = rng.integers(-500, 500, size=Dh).astype(np.int32)
    b2 = rng.integers(-500, 500, size=D).astype(np.int32)
    m1, s1 = api.channel_requant_prepare((2047 / (4 * 74.0 * 4.6 * np.sqrt(D))) * 2.0 ** rng.uniform(-0.3, 0.3, size=Dh))
    m2, s2 = api.channel_requant_prepare(2.0 ** rng.uniform(-9, -7, size=D))
    go, ga = orc.gelu_prepare(4.0 / 2047, 12, 0.03, -100, 8, 0), api.gelu_prepare(4.0 / 2047, 12, 0.03, -100, 8, 0)
    p1, p2 = synth.pack_int4(w1), synth.pack_int4(w2)
    res = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    rro, rra = orc.requant_prepare(0.5 / 65536), api.requant_prepare(0.5 / 65536)
    ws = api.Workspace(api.mlp_workspace_bytes(M, D, Dh, 4))
    want_h = orc.mlp_block(x, p1, b1, m1, s1, go, w_bits=4)
    got_h = api.mlp_block(_cu(x), _cu(p1), _cu(b1), _cu(m1), _cu(s1), ga, ws, w_bits=4).cpu().numpy()
    ws.check()
    assert len(np.unique(want_h)) > 30
    assert (got_h == want_h).all(), _mismatch(got_h, want_h)
    want = orc.mlp_block(x, p1, b1, m1, s1, go, p2, b2, m2, s2, 1, res, rro, w_bits=4)
    got = api.mlp_block(_cu(x), _cu(p1), _cu(b1), _cu(m1), _cu(s1), ga, ws, _cu(p2), _cu(b2), _cu(m2), _cu(s2), 1,
                        _cu(res), rra, w_bits=4).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)
    assert (want == orc.mlp_block(x, w1, b1, m1, s1, go, w2, b2, m2, s2, 1, res, rro)).all()


@pytest.mark.parametrize("n,k", [(1, 34), (3, 30), (16, 64), (40, 48), (96, 1536)])
def test_unpack_int4(api, n, k):
    """Every nibble value in every position; sizes that take the 16-byte vector kernel and sizes that fall back to the
    byte-wise one (the expected values are the definition: low nibble first, two's complement)."""
    rng = np.random.default_rng(n * k)
    q = rng.integers(-8, 8, size=(n, k)).astype(np.int8)
    q.reshape(-1)[:16] = np.arange(-8, 8)
    got = api.unpack_int4(_cu(synth.pack_int4(q))).cpu().numpy()
    assert (got == q).all()


def test_linear_errors(api):
    import torch
    ws = api.Workspace(256)
    x = torch.zeros((8, 24), dtype=torch.int8, device="cuda")
    w = torch.zeros((16, 24), dtype=torch.int8, device="cuda")
    m = torch.full((16,), 1 << 30, dtype=torch.int32, device="cuda")
    s = torch.ones((16,), dtype=torch.int8, device="cuda")
    with pytest.raises(api.IptqError) as e:
        api.linear(x, w, None, m, s, ws)          # K not a multiple of 16
    assert e.value.status == api.ERR_SHAPE


@pytest.mark.parametrize("variant", [0, 1, 2])
# hidden widths that are multiples of the 128-channel tile (768, 1536, 384) and one that is not (288)
# (14300, 1536, 1024): FC1 with a reduction long enough, and enough tiles, for CTA pairs (both GELU epilogues on the
# pair kernel)
@pytest.mark.parametrize("M,D,Dh", [(197, 192, 768), (333, 384, 1536), (64, 96, 384), (130, 96, 288), (14300, 1536, 1024)])
def test_mlp_parity(api, orc, variant, M, D, Dh):
    rng = np.random.default_rng(M + variant)
    x = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    w1 = rng.integers(-128, 128, size=(Dh, D)).astype(np.int8)
    b1 = rng.integers(-2000, 2000, size=Dh).astype(np.int32)
    in_bits = 12
    # accumulator std ~ 74*74*sqrt(D); bring 4 sigma to the in_bits range
    acc_std = 74.0 * 74.0 * np.sqrt(D)
    r1 = (2047 / (4 * acc_std)) * 2.0 ** rng.uniform(-0.3, 0.3, size=Dh)
    m1, s1 = api.channel_requant_prepare(r1)
    S_in = 4.0 / 2047                                   # the GELU sees roughly N(0, 1)
    go = orc.gelu_prepare(S_in, in_bits, 0.03, -100, 8, variant)
    ga = api.gelu_prepare(S_in, in_bits, 0.03, -100, 8, variant)
    w2 = rng.integers(-128, 128, size=(D, Dh)).astype(np.int8)
    b2 = rng.integers(-2000, 2000, size=D).astype(np.int32)
    m2, s2 = api.channel_requant_prepare(2.0 ** rng.uniform(-13, -11, size=D))
    res = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    rro, rra = orc.requant_prepare(0.5 / 65536), api.requant_prepare(0.5 / 65536)
    ws = api.Workspace(api.mlp_workspace_bytes(M, D, Dh))
    # stop after GELU
    want_h = orc.mlp_block(x, w1, b1, m1, s1, go)
    got_h = api.mlp_block(_cu(x), _cu(w1), _cu(b1), _cu(m1), _cu(s1), ga, ws).cpu().numpy()
    ws.check()
    assert len(np.unique(want_h)) > 50
    assert (got_h == want_h).all(), _mismatch(got_h, want_h)
    # the same epilogue reading the tabulated GELU instead of evaluating it
    gt = api.gelu_prepare(S_in, in_bits, 0.03, -100, 8, variant)
    tab = api.gelu_table(gt)
    got_t = api.mlp_block(_cu(x), _cu(w1), _cu(b1), _cu(m1), _cu(s1), gt, ws).cpu().numpy()
    ws.check()
    assert (got_t == want_h).all(), _mismatch(got_t, want_h)
    xs = np.arange(-32768, 32768, dtype=np.int32)
    assert (tab.cpu().numpy() == orc.gelu(xs, go)).all()         # the table itself is the oracle's GELU on every input
    # full MLP with residual
    want = orc.mlp_block(x, w1, b1, m1, s1, go, w2, b2, m2, s2, 1, res, rro)
    got = api.mlp_block(_cu(x), _cu(w1), _cu(b1), _cu(m1), _cu(s1), ga, ws, _cu(w2), _cu(b2), _cu(m2), _cu(s2), 1,
                        _cu(res), rra).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
@pytest.mark.parametrize("B,H,N,dh,use_bias,use_mask", [
    (2, 3, 197, 64, False, False), (3, 2, 49, 32, True, False), (4, 3, 49, 32, True, True),
    (1, 1, 1, 64, False, False), (2, 2, 128, 64, False, False), (1, 2, 129, 32, False, False),
    (1, 1, 256, 64, True, False), (2, 1, 80, 32, False, True), (5, 6, 197, 64, False, False),
    # windows (N <= 64, two problems per item): odd problem counts, full and tiny windows, both head dimensions
    (5, 1, 49, 64, True, True), (3, 3, 64, 32, False, False), (2, 3, 16, 32, True, False), (7, 1, 33, 64, False, True),
    (2, 2, 1, 32, False, False), (40, 3, 49, 32, True, True), (1, 2, 64, 64, True, True)])
def test_attention_parity(api, orc, variant, B, H, N, dh, use_bias, use_mask):
    rng = np.random.default_rng(B * 1000 + N + dh + variant)
    q, k, v = (np.clip(np.round(rng.normal(0, 40, size=(B, H, N, dh))), -128, 127).astype(np.int8) for _ in range(3))
    # logit scale: q.k has std ~ 1600 * sqrt(dh); put the logits on N(0, 3^2)
    S = 3.0 / (1600.0 * np.sqrt(dh))
    bias = np.round(rng.normal(0, 1, size=(H, N, N)) / S).astype(np.int32) if use_bias else None
    mask_id = rng.integers(0, 3, size=(B, N)).astype(np.uint8) if use_mask else None
    bits = 4 if variant == 3 else 8                        # the logarithm candidate writes 4-bit codes ...
    ratio = 0.011 / 256 if variant == 3 else 0.011         # ... and accumulates at scale 2^-15 instead of 2^-7
    so, sa = orc.softmax_prepare(S, N, bits, variant), api.softmax_prepare(S, N, bits, variant)
    ro, ra = orc.requant_prepare(ratio, zp=1), api.requant_prepare(ratio, zp=1)
    want = orc.attention_block(q, k, v, so, ro, bias, mask_id)
    ws = api.Workspace(api.attention_workspace_bytes(B, H, N, dh))
    got = api.attention_block(_cu(q), _cu(k), _cu(v), sa, ra, ws, _cu(bias), _cu(mask_id)).cpu().numpy()
    ws.check()
    assert len(np.unique(want)) > 10 or N == 1
    assert (got == want).all(), _mismatch(got, want)
    if use_bias and N <= 64:
        # the same call with the bias laid out once at load time (what an encoder block of a window model does)
        bias_d = _cu(bias)
        bias_t = api.attention_bias_prepare(bias_d)
        assert bias_t is not None
        got = api.attention_block(_cu(q), _cu(k), _cu(v), sa, ra, ws, bias_d, _cu(mask_id), bias_t=bias_t).cpu().numpy()
        ws.check()
        assert (got == want).all(), _mismatch(got, want)


@pytest.mark.parametrize("variant", [0, 2, 3])
@pytest.mark.parametrize("B,H,N,dh,use_mask,table", [(2, 2, 197, 64, False, True), (3, 1, 49, 32, True, True),
                                                      (2, 2, 80, 32, True, False), (1, 3, 130, 64, True, True)])
def test_attention_scores_at_the_bottom_of_the_range(api, orc, variant, B, H, N, dh, use_mask, table):
    """Biased scores close to -2^30 in every row (the lowest the contract admits): padding columns and masked pairs
    must still contribute exactly nothing, with the exponential from the table and evaluated."""
    rng = np.random.default_rng(N + variant)
    q, k, v = (np.clip(np.round(rng.normal(0, 40, size=(B, H, N, dh))), -128, 127).astype(np.int8) for _ in range(3))
    S = 3.0 / (1600.0 * np.sqrt(dh))
    # |q.k| <= 128 * 128 * 64 = 2^20: the bias puts every score within 2^21 + 2^16 of -2^30
    bias = (-(1 << 30) + (1 << 21) + rng.integers(0, 1 << 16, size=(H, N, N))).astype(np.int32)
    mask_id = rng.integers(0, 3, size=(B, N)).astype(np.uint8) if use_mask else None
    bits = 4 if variant == 3 else 8
    ratio = 0.011 / 256 if variant == 3 else 0.011
    so, sa = orc.softmax_prepare(S, N, bits, variant), api.softmax_prepare(S, N, bits, variant)
    keep = api.softmax_table(sa) if table else None
    ro, ra = orc.requant_prepare(ratio, zp=1), api.requant_prepare(ratio, zp=1)
    want = orc.attention_block(q, k, v, so, ro, bias, mask_id)
    ws = api.Workspace(api.attention_workspace_bytes(B, H, N, dh))
    got = api.attention_block(_cu(q), _cu(k), _cu(v), sa, ra, ws, _cu(bias), _cu(mask_id)).cpu().numpy()
    ws.check()
    assert (got == want).all(), _mismatch(got, want)
    del keep


def _oracle_block(orc, spec, table):
    from oracle import compose
    return orc.encoder_block(spec.x, compose.block_params(spec, table))


@pytest.mark.parametrize("shape,w_bits,table", [
    (synth.CONFIGS["cfg0"], 8, (0, 0, 0, 0)),
    (synth.BlockShape("DeiT-S b3", 3, 197, 384, 6, 64, 1536), 8, (0, 0, 0, 0)),
    (synth.BlockShape("DeiT-S b2 alt", 2, 197, 384, 6, 64, 1536), 8, (1, 1, 1, 1)),
    (synth.BlockShape("ViT-B b1 W4", 1, 197, 768, 12, 64, 3072), 4, (2, 2, 1, 0)),
    (synth.BlockShape("Swin-T 8 windows", 8, 49, 96, 3, 32, 384, True), 8, (0, 0, 0, 0)),
    (synth.BlockShape("DeiT-S b2 log2", 2, 197, 384, 6, 64, 1536), 8, (3, 0, 0, 0)),
    (synth.BlockShape("DeiT-T b2 ptf", 2, 197, 192, 3, 64, 768), 8, (1, 0, 2, 2)),
    (synth.BlockShape("Swin-T 8 windows log2", 8, 49, 96, 3, 32, 384, True), 8, (3, 1, 1, 1)),
])
def test_encoder_block_parity(api, orc, shape, w_bits, table):
    _block_parity(api, orc, synth.make_block(shape, seed=1, w_bits=w_bits, gelu_in_bits=14 if table[1] == 2 else 16),
                  w_bits, table)


@pytest.mark.parametrize("shape,table", [
    (synth.BlockShape("DeiT-S b2 W6A6", 2, 197, 384, 6, 64, 1536), (0, 0, 0, 0)),
    (synth.BlockShape("DeiT-T b3 W6A6 alt", 3, 197, 192, 3, 64, 768), (1, 1, 1, 2)),
    (synth.BlockShape("Swin-T 8 windows W6A6", 8, 49, 96, 3, 32, 384, True), (2, 0, 0, 0)),
    (synth.BlockShape("DeiT-S b1 W6A6 log2", 1, 197, 384, 6, 64, 1536), (3, 0, 0, 0)),
])
def test_encoder_block_w6a6_parity(api, orc, shape, table):
    """6-bit weights and activations (the W6A6 column of the object-detection results, Table 8): every operator of the block emits signed 6-bit codes."""
    spec = synth.make_block(shape, seed=2, w_bits=6, a_bits=6)
    _block_parity(api, orc, spec, 6, table)
    y = api.EncoderBlock(spec, table)(_cu(spec.x)).cpu().numpy()
    assert y.min() >= -32 and y.max() <= 31


def _block_parity(api, orc, spec, w_bits, table):
    want = _oracle_block(orc, spec, table)
    blk = api.EncoderBlock(spec, table)
    got = blk(_cu(spec.x)).cpu().numpy()
    blk.ws.check()
    assert len(np.unique(want)) > 30
    assert (got == want).all(), _mismatch(got, want)
    # FC1 epilogue evaluating the polynomial, attention building its exponential table per CTA
    blk2 = api.EncoderBlock(spec, table, gelu_table_on=False, softmax_table_on=False)
    got2 = blk2(_cu(spec.x)).cpu().numpy()
    blk2.ws.check()
    assert (got2 == want).all(), _mismatch(got2, want)
    if w_bits == 4:
        # int4 weights unpacked once at load time instead of at every call
        blk3 = api.EncoderBlock(spec, table, unpack_w4_once=True)
        got3 = blk3(_cu(spec.x)).cpu().numpy()
        blk3.ws.check()
        assert (got3 == want).all(), _mismatch(got3, want)
        wq = spec.qkv
        assert (api.unpack_int4(_cu(wq.w_packed)).cpu().numpy() == wq.w).all()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_workspace_recovers(api, orc):
    """A wait nothing ever satisfies (the self-test kernel waits on a barrier without arrivals) gives up after the
    workspace's limit, records itself, and the kernel returns: iptq_check reports the time-out, and the same
    workspace runs an ordinary layer bit-exactly after it has been re-initialised."""
    rng = np.random.default_rng(77)
    M, N, K = 300, 256, 128
    x, w, bias, ratios = _linear_case(rng, M, N, K)
    ma, sa = api.channel_requant_prepare(ratios)
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K))
    ws.set_wait_limit(1000)                                     # 1 ms instead of 2 s
    assert api.lib().iptq_selftest_wait_timeout(ws.ptr, ws.nbytes, None) == api.OK
    with pytest.raises(api.IptqError) as e:
        ws.check()
    assert e.value.status == api.ERR_TIMEOUT
    flag, where, block, work_next, work_done, limit = ws.status_words()
    assert flag == 1 and where == 99 and block == 0 and work_next == 0 and work_done == 0 and limit == 1000
    ws.reset()
    assert ws.status_words()[:3] == [0, 0, 0]
    got = api.linear(_cu(x), _cu(w), _cu(bias), _cu(ma), _cu(sa), ws, out_zp=3).cpu().numpy()
    ws.check()
    assert (got == orc.linear(x, w, bias, ma, sa, out_zp=3)).all()


def test_the_plan_for_the_current_device_is_the_plan_that_runs(api):
    """`linear_plan` with sm_count = 0 reads the device; on the part this library targets that is 148 SMs."""
    import torch
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for shape in [(25216, 2304, 768), (25216, 768, 3072), (12608, 384, 1536), (197, 192, 192)]:
        here, given = api.linear_plan(*shape, residual=True), api.linear_plan(*shape, residual=True, sm_count=sms)
        assert [getattr(here, f) for f, _ in here._fields_] == [getattr(given, f) for f, _ in given._fields_]
