"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every function that
include/iptq.h declares, and its host-side *_prepare functions and argument checks (which touch no
device) agree with the oracle's own constant preparation."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2511_15369_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2511_15369_b200 import api as _api
    from paper_2511_15369_b200 import build
    build.build()
    _api.lib()
    return _api


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "iptq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(iptq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_function_is_exported(api):
    names = _declared_functions()
    assert len(names) >= 20
    L = api.lib()
    for n in names:
        assert getattr(L, n) is not None, n
    assert sorted(api.exported_symbols()) == names


def test_no_torch_types_in_the_header():
    text = open(os.path.join(ROOT, "include", "iptq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    assert "torch" not in text and "at::" not in text and "Tensor" not in text and "#include <cuda" not in text


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("scale,n", [(synth.SOFTMAX_SCALE_ACC, 197), (synth.SOFTMAX_SCALE_8BIT, 49), (1 / 255.5, 1)])
def test_softmax_constants_match_the_oracle(api, orc, variant, scale, n):
    a, o = api.softmax_prepare(scale, n, 8, variant), orc.softmax_prepare(scale, n, 8, variant)
    for f, _ in o._fields_:
        assert getattr(a, f) == getattr(o, f), f
    # the derived magic divisor reproduces floor(v / divisor) on the whole range the kernels use
    div = a.qln2 if variant == 2 else a.x0
    v = np.concatenate([np.arange(0, 70000), np.random.default_rng(0).integers(0, 2 ** 31, 200000)]).astype(np.uint64)
    q = ((v * np.uint64(a.div_mul)) >> np.uint64(32)) >> np.uint64(a.div_shift)
    assert (q == v // np.uint64(div)).all()


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_gelu_and_layernorm_constants_match_the_oracle(api, orc, variant):
    bits, S = (16, 1.3e-4) if variant != 2 else (12, 0.003)
    a, o = api.gelu_prepare(S, bits, 0.03, -7, 8, variant), orc.gelu_prepare(S, bits, 0.03, -7, 8, variant)
    for f, t in o._fields_:
        if f == "out":
            for g, _ in a.out._fields_:
                assert getattr(a.out, g) == getattr(o.out, g), g
        else:
            assert getattr(a, f) == getattr(o, f), f
    _, gamma, beta, _ = synth.ln_values(4, 192, seed=3)
    ga, ba, ca = api.layernorm_prepare(gamma, beta, 0.02, 3, 8, variant)
    go, bo, co = orc.layernorm_prepare(gamma, beta, 0.02, 3, 8, variant)
    assert (ga == go).all() and (ba == bo).all()
    assert (ca.out.mult, ca.out.shift, ca.out.zp, ca.out.qmin, ca.out.qmax) == \
           (co.out.mult, co.out.shift, co.out.zp, co.out.qmin, co.out.qmax)


def test_requant_prepare_matches_the_oracle_and_rejects_bad_ratios(api, orc):
    rng = np.random.default_rng(1)
    for r in 2.0 ** rng.uniform(-33, -2.001, size=300):
        a, o = api.requant_prepare(r, 2), orc.requant_prepare(r, 2)
        assert (a.mult, a.shift, a.zp) == (o.mult, o.shift, o.zp)
    for bad in (0.25, 0.3, 1.0, 0.0, -1.0, 2.0 ** -40):
        with pytest.raises(api.IptqError) as e:
            api.requant_prepare(bad)
        assert e.value.status == api.ERR_SCALE_RANGE
    m, s = api.channel_requant_prepare(np.array([2.0 ** -9, 0.2]))
    assert m.dtype == np.int32 and s.tolist() == [orc.requant_prepare(2.0 ** -9).shift, orc.requant_prepare(0.2).shift]


def test_argument_errors_are_reported_before_any_launch(api):
    """These calls fail on the host-side checks, so they run without a device."""
    L = api.lib()
    c = api.softmax_prepare(synth.SOFTMAX_SCALE_ACC, 197)
    assert L.iptq_softmax(None, None, 4, 197, None, 1, None, None) == api.ERR_NULL
    assert L.iptq_softmax(None, None, 4, 49, None, 1, C.byref(c), None) == api.ERR_SHAPE      # row_len != consts
    assert L.iptq_softmax(None, None, 4, 197, None, 1, C.byref(c), None) == api.ERR_NULL      # null tensors
    assert L.iptq_softmax(None, None, 0, 197, None, 1, C.byref(c), None) == api.OK            # empty input
    assert L.iptq_softmax(16, 24, 4, 197, None, 1, C.byref(c), None) == api.ERR_ALIGN
    g = api.gelu_prepare(1.3e-4, 16, 0.03, 0)
    assert L.iptq_gelu(None, None, 0, C.byref(g), None) == api.OK
    assert L.iptq_gelu(None, None, 5, C.byref(g), None) == api.ERR_NULL
    assert L.iptq_gelu(None, None, -1, C.byref(g), None) == api.ERR_SHAPE
    with pytest.raises(api.IptqError) as e:
        api.gelu_prepare(1.3e-4, 17, 0.03, 0)
    assert e.value.status == api.ERR_BITS
    with pytest.raises(api.IptqError) as e:
        api.softmax_prepare(0.5, 197)
    assert e.value.status == api.ERR_SCALE_RANGE
    with pytest.raises(api.IptqError) as e:
        api.softmax_prepare(synth.SOFTMAX_SCALE_ACC, 197, 8, 7)
    assert e.value.status == api.ERR_VARIANT
    assert L.iptq_linear(None, None, 5, None, None, None, 0, None, None, None, 8, 16, 16, None, 0, None) == api.ERR_BITS
    assert L.iptq_linear(None, None, 8, None, None, None, 0, None, None, None, 8, 16, 16, None, 0, None) == api.ERR_WORKSPACE
    assert L.iptq_attention_block(None, None, None, None, 1, 1, 49, 32, None, None, None, None, None, None, 0, None) \
        == api.ERR_WORKSPACE
    # a rejected call with packed 4-bit weights has launched nothing, the unpack kernel included
    n0 = L.iptq_launch_count()
    fake = 4096                                               # a non-NULL, 256-byte aligned stand-in: never dereferenced
    assert L.iptq_linear(None, fake, 4, None, fake, fake, 0, None, None, fake, 8, 16, 16, fake, 1 << 20, None) == api.ERR_NULL
    assert L.iptq_linear(fake, fake, 4, None, fake, fake, 0, None, None, fake, 8, 24, 16, fake, 1 << 20, None) == api.ERR_SHAPE
    g2 = api.gelu_prepare(1.3e-4, 16, 0.03, 0)
    assert L.iptq_mlp_block(fake, fake, None, fake, fake, C.byref(g2), fake, None, None, fake, 0, None, None, fake,
                            8, 16, 64, 4, fake, 1 << 20, None) == api.ERR_NULL    # FC2's multiplier is missing
    assert L.iptq_launch_count() == n0
    assert api.lib().iptq_strerror(api.ERR_TIMEOUT).decode() != ""
    assert api.linear_workspace_bytes(100, 256, 384, 4) >= 256 + 256 * 384
    assert api.mlp_workspace_bytes(100, 384, 1536) >= 256 + 100 * 1536
