"""Guard bytes round every GPU output: each output tensor of a call sits between two 256-byte fences filled with a
pattern, and the fences must be untouched after the call (the stand-in for a memory checker: a kernel that writes
one row or one tile too far would land there and, without the fences, in a neighbouring allocation where no test
looks).  Shapes are chosen off the tile sizes: token counts that are no multiple of a tile, channel counts that end
inside a 128-channel tile, 197 / 129 / 1 tokens for the attention."""
import numpy as np
import pytest

from paper_2511_15369_b200 import synth

pytestmark = pytest.mark.gpu
FENCE = 256
PATTERN = 0xA5


@pytest.fixture(scope="module")
def api():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2511_15369_b200 import api as _api
    _api.lib()
    return _api


class Guarded:
    """An int8 / uint8 device tensor of `shape` with FENCE pattern bytes in front of it and behind it."""

    def __init__(self, shape, dtype=None):
        import torch
        self.n = int(np.prod(shape))
        pad = (-self.n) % 16
        self.buf = torch.full((FENCE + self.n + pad + FENCE,), PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.buf[FENCE:FENCE + self.n].view(dtype or torch.int8).view(*shape)
        assert self.t.data_ptr() % 16 == 0

    def check(self):
        import torch
        torch.cuda.synchronize()
        front = self.buf[:FENCE]
        back = self.buf[FENCE + self.n:]
        assert bool((front == PATTERN).all()), "bytes in front of the output were overwritten"
        assert bool((back == PATTERN).all()), "bytes behind the output were overwritten"


def _cu(a):
    import torch
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


# (7090, 2064, 1536): CTA pairs, ragged last channel tile in the odd CTA's half, ragged last token tile
@pytest.mark.parametrize("M,N,K", [(197, 144, 96), (333, 1008, 768), (5, 16, 16), (130, 400, 272), (257, 384, 1536),
                                   (7090, 2064, 1536)])
def test_linear_outputs_stay_inside_their_tensor(api, orc, M, N, K):
    rng = np.random.default_rng(M + N)
    x = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    w = rng.integers(-128, 128, size=(N, K)).astype(np.int8)
    bias = rng.integers(-3000, 3000, size=N).astype(np.int32)
    ma, sa = api.channel_requant_prepare(2.0 ** rng.uniform(-12, -7, size=N))
    res = rng.integers(-128, 128, size=(M, N)).astype(np.int8)
    rro, rra = orc.requant_prepare(0.9 / 65536, zp=-4), api.requant_prepare(0.9 / 65536, zp=-4)
    ws = api.Workspace(api.linear_workspace_bytes(M, N, K))
    for residual in (False, True):
        out = Guarded((M, N))
        api.linear(_cu(x), _cu(w), _cu(bias), _cu(ma), _cu(sa), ws, out_zp=2, residual=_cu(res) if residual else None,
                   residual_rq=rra if residual else None, out=out.t)
        ws.check()
        out.check()
        want = orc.linear(x, w, bias, ma, sa, out_zp=2, residual=res if residual else None,
                          residual_rq=rro if residual else None)
        assert (out.t.cpu().numpy() == want).all()


def test_mlp_outputs_stay_inside_their_tensor(api, orc):
    rng = np.random.default_rng(9)
    M, D, Dh = 203, 96, 384
    x = rng.integers(-128, 128, size=(M, D)).astype(np.int8)
    w1 = rng.integers(-128, 128, size=(Dh, D)).astype(np.int8)
    b1 = rng.integers(-500, 500, size=Dh).astype(np.int32)
    m1, s1 = api.channel_requant_prepare((2047 / (64 * 74.0 * 4.6 * np.sqrt(D))) * 2.0 ** rng.uniform(-0.3, 0.3, size=Dh))
    go, ga = orc.gelu_prepare(4.0 / 2047, 12, 0.03, -100, 8, 0), api.gelu_prepare(4.0 / 2047, 12, 0.03, -100, 8, 0)
    want = orc.mlp_block(x, w1, b1, m1, s1, go)
    for table in (False, True):
        keep = api.gelu_table(ga) if table else None
        ws = api.Workspace(api.mlp_workspace_bytes(M, D, Dh))
        out = Guarded((M, Dh))
        api.mlp_block(_cu(x), _cu(w1), _cu(b1), _cu(m1), _cu(s1), ga, ws, out=out.t)
        ws.check()
        out.check()
        assert (out.t.cpu().numpy() == want).all()
        del keep


@pytest.mark.parametrize("B,H,N,dh,use_bias", [(2, 3, 197, 64, False), (1, 2, 129, 32, False), (3, 1, 1, 64, False),
                                               (5, 3, 49, 32, True), (1, 1, 256, 64, True)])
def test_attention_outputs_stay_inside_their_tensor(api, orc, B, H, N, dh, use_bias):
    rng = np.random.default_rng(B + N)
    q, k, v = (np.clip(np.round(rng.normal(0, 40, size=(B, H, N, dh))), -128, 127).astype(np.int8) for _ in range(3))
    S = 3.0 / (1600.0 * np.sqrt(dh))
    bias = np.round(rng.normal(0, 1, size=(H, N, N)) / S).astype(np.int32) if use_bias else None
    so, sa = orc.softmax_prepare(S, N), api.softmax_prepare(S, N)
    ro, ra = orc.requant_prepare(0.011, zp=1), api.requant_prepare(0.011, zp=1)
    ws = api.Workspace(api.attention_workspace_bytes(B, H, N, dh))
    out = Guarded((B, N, H * dh))
    api.attention_block(_cu(q), _cu(k), _cu(v), sa, ra, ws, _cu(bias), out=out.t)
    ws.check()
    out.check()
    assert (out.t.cpu().numpy() == orc.attention_block(q, k, v, so, ro, bias)).all()


def test_rowwise_kernels_and_gather_stay_inside_their_tensors(api, orc):
    import torch
    rng = np.random.default_rng(3)
    # Softmax: 197 uint8 per row, rows of odd length
    s = synth.quantize_scores(synth.softmax_logits(77, 197, seed=1), synth.SOFTMAX_SCALE_ACC)
    out = Guarded((77, 197), torch.uint8)
    api.softmax(_cu(s), api.softmax_prepare(synth.SOFTMAX_SCALE_ACC, 197), out=out.t)
    out.check()
    assert (out.t.cpu().numpy() == orc.softmax(s, orc.softmax_prepare(synth.SOFTMAX_SCALE_ACC, 197))).all()
    # GELU: a length that is no multiple of the vector width
    x, S = synth.quantize_sym(synth.gelu_values(4099, seed=2), 16)
    So, zp = synth.affine_out_quant(synth.gelu_ref(x[:4096] * S))
    out = Guarded((4099,))
    api.gelu(_cu(x), api.gelu_prepare(S, 16, So, zp), out=out.t)
    out.check()
    assert (out.t.cpu().numpy() == orc.gelu(x, orc.gelu_prepare(S, 16, So, zp))).all()
    # LayerNorm: general and short-row kernels
    for rows, dim in ((203, 192), (1001, 96)):
        xf, gamma, beta, _ = synth.ln_values(rows, dim, seed=4)
        xq, _ = synth.quantize_sym(xf, 8, np.int8)
        So, zp = synth.affine_out_quant(synth.layernorm_ref(xq.astype(np.float64), gamma, beta))
        gq, bq, lc = api.layernorm_prepare(gamma, beta, So, zp)
        go, bo, lo = orc.layernorm_prepare(gamma, beta, So, zp)
        out = Guarded((rows, dim))
        api.layernorm(_cu(xq), _cu(gq), _cu(bq), lc, out=out.t)
        out.check()
        assert (out.t.cpu().numpy() == orc.layernorm(xq, go, bo, lo)).all()
    # row gather
    src = rng.integers(-128, 128, size=(500, 96)).astype(np.int8)
    idx = rng.integers(-1, 500, size=(333, 4)).astype(np.int32)
    out = Guarded((333, 4 * 96))
    api.gather_rows(_cu(src), _cu(idx), out=out.t)
    out.check()


def test_encoder_block_output_stays_inside_its_tensor(api, orc):
    from oracle import compose
    spec = synth.make_block(synth.BlockShape("DeiT-S b3", 3, 197, 384, 6, 64, 1536), seed=5)
    table = (0, 0, 0, 0)
    blk = api.EncoderBlock(spec, table)
    out = Guarded(spec.x.shape)
    blk(_cu(spec.x), out.t)
    blk.ws.check()
    out.check()
    assert (out.t.cpu().numpy() == orc.encoder_block(spec.x, compose.block_params(spec, table))).all()
