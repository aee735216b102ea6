"""GPU parity of the stand-alone integer Softmax / GELU / LayerNorm kernels: bit-exact against the
CPU oracle on the same seeded inputs, through the C-ABI."""
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
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_prepared_constants_agree_with_the_oracle(api, orc):
    for S in (3e-4, 12 / 127, 1 / 777.7):
        for n in (1, 49, 197, 1024):
            for var in (0, 1, 2):
                a, b = api.softmax_prepare(S, n, 8, var), orc.softmax_prepare(S, n, 8, var)
                for f, _ in b._fields_:
                    assert getattr(a, f) == getattr(b, f), (f, S, n, var)
    for S, bits in ((1.3e-4, 16), (2e-3, 12), (0.05, 8)):
        for var in (0, 1, 2):
            a, b = api.gelu_prepare(S, bits, 0.02, -100, 8, var), orc.gelu_prepare(S, bits, 0.02, -100, 8, var)
            for f, _ in b._fields_[:-1]:
                assert getattr(a, f) == getattr(b, f), (f, S, bits, var)
            for f in ("mult", "shift", "zp", "qmin", "qmax"):
                assert getattr(a.out, f) == getattr(b.out, f)
    rng = np.random.default_rng(0)
    for r in 2.0 ** rng.uniform(-32, -2.001, size=200):
        a, b = api.requant_prepare(r), orc.requant_prepare(r)
        assert (a.mult, a.shift) == (b.mult, b.shift)


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("rows,n", [(591, 197), (1000, 49), (33, 1), (17, 2), (40, 208), (9, 1000), (5, 64)])
@pytest.mark.parametrize("scale", [synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT])
def test_softmax_parity(api, orc, variant, rows, n, scale):
    s = synth.quantize_scores(synth.softmax_logits(rows, n, seed=rows + n), scale)
    want = orc.softmax(s, orc.softmax_prepare(scale, n, 8, variant))
    got = api.softmax(_cu(s), api.softmax_prepare(scale, n, 8, variant)).cpu().numpy()
    assert (got == want).all()


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
@pytest.mark.parametrize("scale", [synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT])
@pytest.mark.parametrize("rows,n,use_table", [(6001, 197, True), (86017, 197, False), (86017, 197, True),
                                              (40003, 49, True), (9000, 208, True)])
def test_softmax_tabulated_parity(api, orc, variant, scale, rows, n, use_table):
    """Inputs large enough for the kernel that reads the exponential from a shared-memory table, with the table
    copied from device memory (iptq_softmax_table) or built by every CTA."""
    base = 4096
    s0 = synth.quantize_scores(synth.softmax_logits(base, n, seed=rows + n), scale)
    s0[7] = -(1 << 30) + 1
    s0[7, n // 2] = (1 << 30) - 1                  # largest admissible distance to the row maximum
    s0[8] = 12345                                  # all-equal row
    s0[9] = -(1 << 30) + 3001                      # every entry at the bottom of the admissible range (bias included)
    s0[10] = -(1 << 30) + 3001 + np.arange(n) * 7
    reps = (rows + base - 1) // base
    s = np.ascontiguousarray(np.tile(s0, (reps, 1))[:rows])
    bias = np.random.default_rng(5).integers(-3000, 3000, size=(3, n)).astype(np.int32)
    bits = 4 if variant == 3 else 8
    co = orc.softmax_prepare(scale, n, bits, variant)
    ca = api.softmax_prepare(scale, n, bits, variant)
    keep = api.softmax_table(ca) if use_table else None
    assert (keep is not None) == use_table and bool(ca.table) == use_table
    want0 = orc.softmax(s0, co)
    got = api.softmax(_cu(s), ca).cpu().numpy()
    assert (got == np.tile(want0, (reps, 1))[:rows]).all()
    sub = slice(rows - 1500, rows)                 # rows whose bias row differs from their position in the block
    want_b = orc.softmax(np.ascontiguousarray(s[sub]), co,
                         bias=np.ascontiguousarray(np.roll(bias, -((rows - 1500) % 3), axis=0)), bias_period=3)
    got_b = api.softmax(_cu(s), ca, bias=_cu(bias)).cpu().numpy()
    assert (got_b[sub] == want_b).all()


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
@pytest.mark.parametrize("scale,n", [(synth.SOFTMAX_SCALE_ACC, 197), (synth.SOFTMAX_SCALE_8BIT, 197), (1.0 / 700, 49)])
def test_softmax_table_contents(api, orc, variant, scale, n):
    """The device table holds the oracle's exponential for every tabulated distance, and the oracle's
    exponential is 0 at every distance the table leaves out (up to the clamp of Eq. (6))."""
    bits = 4 if variant == 3 else 8
    co = orc.softmax_prepare(scale, n, bits, variant)
    ca = api.softmax_prepare(scale, n, bits, variant)
    t = api.softmax_table(ca)
    assert t is not None and 0 < ca.table_n < api.SOFTMAX_TABLE_MAX
    tab = t.cpu().numpy().view(np.uint16)
    want = np.array([orc.softmax_exp(d, co) for d in range(ca.table_n)])
    assert (tab[:ca.table_n] == want).all()
    assert tab[ca.table_n] == 0
    assert tab[0] == (co.x0 << co.nsh if variant < 2 else orc.softmax_exp(0, co))
    for d in list(range(ca.table_n, min(co.dcap, ca.table_n + 5000))) + list(range(ca.table_n, co.dcap + 1, 97)) + [co.dcap]:
        assert orc.softmax_exp(d, co) == 0, d


def test_softmax_table_absent(api):
    import torch
    c = api.softmax_prepare(1.0 / 8000.5, 49, 8, 2)                   # polynomial exponential, table too long
    assert api.softmax_table(c) is None and not c.table and c.table_n == 0
    c = api.softmax_prepare(1.0 / ((1 << 20) - 2.5), 49)               # x0 too large for a shared-memory table
    assert api.softmax_table(c) is None and not c.table
    c = api.softmax_prepare(synth.SOFTMAX_SCALE_ACC, 197)
    small = torch.empty(64, dtype=torch.int16, device="cuda")
    rc = api.lib().iptq_softmax_table(api.C.byref(c), small.data_ptr(), 64, None)
    assert rc == api.ERR_SHAPE and not c.table


@pytest.mark.parametrize("rows,n", [(591, 197), (1000, 49), (33, 1), (17, 2), (9, 1000), (5000, 64)])
@pytest.mark.parametrize("scale", [synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT])
def test_softmax_log2_parity(api, orc, rows, n, scale):
    """Logarithm candidate: 4-bit power-of-two codes (255 = probability 0), with and without bias."""
    s = synth.quantize_scores(synth.softmax_logits(rows, n, seed=rows + n), scale)
    s[0] = 3                                                  # all-equal row
    if n > 2:
        s[1] = -(1 << 30) + 1
        s[1, 1] = (1 << 30) - 1                               # everything but one entry vanishes
    co = orc.softmax_prepare(scale, n, 4, orc.SM_LOG2)
    ca = api.softmax_prepare(scale, n, 4, api.SM_LOG2)
    want = orc.softmax(s, co)
    got = api.softmax(_cu(s), ca).cpu().numpy()
    assert (got == want).all()
    assert ((got <= 15) | (got == api.LOG2_ZERO)).all()
    bias = np.random.default_rng(1).integers(-2000, 2000, size=(4, n)).astype(np.int32)
    got_b = api.softmax(_cu(s), ca, bias=_cu(bias)).cpu().numpy()
    assert (got_b == orc.softmax(s, co, bias=bias, bias_period=4)).all()
    with pytest.raises(api.IptqError) as e:
        api.softmax_prepare(scale, n, 8, api.SM_LOG2)
    assert e.value.status == api.ERR_BITS


@pytest.mark.parametrize("n", [197, 49, 1000, 1])
@pytest.mark.parametrize("variant", [0, 1, 2, 3])
def test_softmax_rows_at_the_bottom_of_the_range(api, orc, variant, n):
    """Rows whose every entry sits at -2^30 + 1 (the lowest admissible score), with and without a bias: lanes past
    the row end must contribute nothing although the row maximum is as low as a score can be.  Small inputs take
    the evaluated kernel, large ones the tabulated kernel (table built per CTA and copied from device memory)."""
    lo = -(1 << 30) + 1
    bits = 4 if variant == 3 else 8
    for scale in (synth.SOFTMAX_SCALE_ACC, synth.SOFTMAX_SCALE_8BIT):
        co = orc.softmax_prepare(scale, n, bits, variant)
        ca = api.softmax_prepare(scale, n, bits, variant)
        block = np.full((64, n), lo, dtype=np.int32)
        block[1::2] += np.random.default_rng(n).integers(0, 5000, size=(32, n)).astype(np.int32)
        bias = np.random.default_rng(2).integers(0, 4000, size=(4, n)).astype(np.int32)
        want, want_b = orc.softmax(block, co), orc.softmax(block, co, bias=bias, bias_period=4)
        assert (api.softmax(_cu(block), ca).cpu().numpy() == want).all()
        assert (api.softmax(_cu(block), ca, bias=_cu(bias)).cpu().numpy() == want_b).all()
        if n <= 256:
            reps = ((17 << 20) // (64 * n)) + 1                     # past the size where every CTA builds the table
            big = _cu(np.tile(block, (reps, 1)))
            assert (api.softmax(big, ca).cpu().numpy() == np.tile(want, (reps, 1))).all()
            keep = api.softmax_table(ca)
            assert (api.softmax(big, ca).cpu().numpy() == np.tile(want, (reps, 1))).all()
            assert (api.softmax(big, ca, bias=_cu(bias)).cpu().numpy() == np.tile(want_b, (reps, 1))).all()
            del keep


def test_softmax_edge_rows_and_bias(api, orc):
    n = 197
    rng = np.random.default_rng(3)
    s = rng.integers(-50000, 50000, size=(64, n)).astype(np.int32)
    s[0] = 7                                   # all-equal row
    s[1] = -(1 << 30) + 1
    s[1, 5] = (1 << 30) - 1                    # one huge outlier, extreme magnitudes
    s[2] = (1 << 30) - 1
    s[3, :] = np.arange(n) * 1000
    bias = rng.integers(-20000, 20000, size=(3, n)).astype(np.int32)
    for variant in (0, 1, 2):
        for bits in (8, 6, 4):
            co = orc.softmax_prepare(3e-4, n, bits, variant)
            ca = api.softmax_prepare(3e-4, n, bits, variant)
            assert (api.softmax(_cu(s), ca).cpu().numpy() == orc.softmax(s, co)).all()
            got = api.softmax(_cu(s), ca, bias=_cu(bias)).cpu().numpy()
            assert (got == orc.softmax(s, co, bias=bias, bias_period=3)).all()
    # large x0 (N = 0, M capped)
    S = 1.0 / ((1 << 20) - 2.5)
    s2 = rng.integers(-(1 << 26), 1 << 26, size=(32, 49)).astype(np.int32)
    assert (api.softmax(_cu(s2), api.softmax_prepare(S, 49)).cpu().numpy() == orc.softmax(s2, orc.softmax_prepare(S, 49))).all()


def test_softmax_empty_and_errors(api):
    import torch
    c = api.softmax_prepare(3e-4, 197)
    out = api.softmax(torch.empty((0, 197), dtype=torch.int32, device="cuda"), c)
    assert out.shape == (0, 197)
    with pytest.raises(api.IptqError) as e:
        api.softmax(torch.zeros((4, 49), dtype=torch.int32, device="cuda"), c)      # row_len mismatch
    assert e.value.status == api.ERR_SHAPE
    with pytest.raises(api.IptqError) as e:
        api.softmax_prepare(0.5, 197)
    assert e.value.status == api.ERR_SCALE_RANGE


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("n", [151296, 4099, 3, 1 << 20])
def test_gelu_parity(api, orc, variant, n):
    bits = 16 if variant != 2 else 12
    # scales are calibrated on at least 4096 draws so that the ragged n = 3 case keeps a realistic output range
    xall, S = synth.quantize_sym(synth.gelu_values(max(n, 4096), seed=n), bits)
    x = np.ascontiguousarray(xall[:n])
    ref = synth.gelu_ref(xall[:4096] * S)
    So, zp = synth.affine_out_quant(ref)
    want = orc.gelu(x, orc.gelu_prepare(S, bits, So, zp, 8, variant))
    got = api.gelu(_cu(x), api.gelu_prepare(S, bits, So, zp, 8, variant)).cpu().numpy()
    assert (got == want).all()


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("n", [(1 << 20) + 3, 3 * (1 << 20)])
def test_gelu_tabulated_standalone(api, orc, variant, n):
    """iptq_gelu with the table attached (inputs of 2^20 elements and more): values beyond 16 bits included."""
    bits = 16 if variant != 2 else 12
    xall, S = synth.quantize_sym(synth.gelu_values(1 << 16, seed=n + variant), bits)
    x = np.tile(xall, (n + xall.size - 1) // xall.size)[:n].astype(np.int32)
    x[:8] = [-(1 << 31), (1 << 31) - 1, -32769, 32768, -32768, 32767, 0, -1]
    So, zp = synth.affine_out_quant(synth.gelu_ref(xall[:4096] * S))
    want = orc.gelu(x, orc.gelu_prepare(S, bits, So, zp, 8, variant))
    c = api.gelu_prepare(S, bits, So, zp, 8, variant)
    keep = api.gelu_table(c)
    assert (api.gelu(_cu(x), c).cpu().numpy() == want).all()


@pytest.mark.parametrize("bits,S,rng_", [(16, 1.3e-4, (-3.0, 3.0)), (14, 2.0 / 8191, (-1.4, 1.4)), (8, 8.0 / 127, (-5.0, 2.0))])
def test_gelu_refitted_coefficients_exhaustive(api, orc, bits, S, rng_):
    """Quartic GELU with coefficients refitted to a data range (Eq. (4)): every in_bits input and the clamp,
    stand-alone kernel and tabulated form."""
    a, b, _ = api.gelu_fit(rng_[0], rng_[1])
    ca = api.gelu_prepare_coeffs(S, bits, 0.03, -7, 8, a, b)
    co = orc.gelu_prepare_coeffs(S, bits, 0.03, -7, 8, a, b)
    x = np.arange(-(1 << 17), 1 << 17, dtype=np.int32)
    want = orc.gelu(x, co)
    assert (api.gelu(_cu(x), ca).cpu().numpy() == want).all()
    tab = api.gelu_table(ca).cpu().numpy()
    assert (tab == want[(1 << 17) - 32768:(1 << 17) + 32768]).all()


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("bits,S", [(8, 8.0 / 127), (12, 0.003), (16, 1.3e-4)])
def test_gelu_exhaustive_inputs(api, orc, variant, bits, S):
    if variant == 2 and bits == 16:
        S = 1.0 / 9000                     # the shift exponential needs floor(1/S) < 2^14
    x = np.arange(-(1 << 17), 1 << 17, dtype=np.int32)       # covers every in_bits value and the clamp
    for out_bits in (8, 5):
        want = orc.gelu(x, orc.gelu_prepare(S, bits, 0.03, -7, out_bits, variant))
        got = api.gelu(_cu(x), api.gelu_prepare(S, bits, 0.03, -7, out_bits, variant)).cpu().numpy()
        assert (got == want).all()


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("rows,dim", [(197, 192), (300, 384), (100, 768), (513, 96), (7, 1536), (3, 3072), (5, 8)])
def test_layernorm_parity(api, orc, variant, rows, dim):
    xf, gamma, beta, _ = synth.ln_values(rows, dim, seed=dim)
    xq, _ = synth.quantize_sym(xf, 8, np.int8)
    ptf = synth.ptf_shifts(xq) if variant == 2 else None
    ref = synth.layernorm_ref(xq[:64].astype(np.float64), gamma, beta)
    So, zp = synth.affine_out_quant(ref)
    gq, bq, co = orc.layernorm_prepare(gamma, beta, So, zp, 8, variant)
    gq2, bq2, ca = api.layernorm_prepare(gamma, beta, So, zp, 8, variant)
    assert (gq == gq2).all() and (bq == bq2).all()
    assert (ca.out.mult, ca.out.shift, ca.out.zp) == (co.out.mult, co.out.shift, co.out.zp)
    want = orc.layernorm(xq, gq, bq, co, ptf)
    got = api.layernorm(_cu(xq), _cu(gq2), _cu(bq2), ca, None if ptf is None else _cu(ptf)).cpu().numpy()
    assert (got == want).all()


@pytest.mark.parametrize("dim,rows", [(192, 40), (96, 75), (128, 64), (16, 100), (48, 333), (64, 201), (32, 129)])
def test_layernorm_degenerate_rows(api, orc, dim, rows):
    """Constant rows, extreme variances, a ragged last step -- for the general kernel (dim 192) and for the
    four-lanes-per-row kernel of short rows (dim <= 128, at least 64 rows)."""
    rng = np.random.default_rng(5)
    x = rng.integers(-128, 128, size=(rows, dim)).astype(np.int8)
    x[0] = 0
    x[1] = 127                                  # zero variance
    x[2] = -128
    x[3] = 0
    x[3, dim // 2] = 1                          # smallest non-zero variance
    x[4, ::2] = 127
    x[4, 1::2] = -128                           # largest variance
    # rows whose D^2 var + 1 is a perfect square make the fixed-step square root stop one above
    x[5] = 0
    x[5, :3] = [1, 1, 1]
    gamma = rng.normal(1, 0.1, dim).astype(np.float32)
    beta = rng.normal(0, 0.1, dim).astype(np.float32)
    for variant in (0, 1, 2):
        for out_bits, zp in ((8, 3), (6, -2)):
            ptf = synth.ptf_shifts(x) if variant == 2 else None
            gq, bq, co = orc.layernorm_prepare(gamma, beta, 0.02 * (1 << (8 - out_bits)), zp, out_bits, variant)
            _, _, ca = api.layernorm_prepare(gamma, beta, 0.02 * (1 << (8 - out_bits)), zp, out_bits, variant)
            got = api.layernorm(_cu(x), _cu(gq), _cu(bq), ca, None if ptf is None else _cu(ptf)).cpu().numpy()
            assert (got == orc.layernorm(x, gq, bq, co, ptf)).all()
