"""Swin-shaped backbone (config 4): shifted 7x7 windows with padding, relative-position bias, attention labels and
2x2 patch merging, composed from the library's C-ABI calls, against the same composition of CPU-oracle calls
(numpy index gathers for the layout steps).  Bit-exact."""
import numpy as np
import pytest

from paper_2511_15369_b200 import synth
from test_gpu_blocks import _oracle_block

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2511_15369_b200 import api as _api
    _api.lib()
    return _api


def _gather(src, index):
    index = index.reshape(-1) if index.ndim == 1 else index
    if index.ndim == 1:
        index = index[:, None]
    parts = [np.where(index[:, p:p + 1] >= 0, src[np.maximum(index[:, p], 0)], 0) for p in range(index.shape[1])]
    return np.ascontiguousarray(np.concatenate(parts, axis=1).astype(np.int8))


def _oracle_backbone(orc, spec, table):
    x = spec.x
    for st in spec.stages:
        for bspec, shift, fwd, rev in st["blocks"]:
            bspec.x = _gather(x, fwd)
            yw = _oracle_block(orc, bspec, table)
            bspec.x = None
            x = _gather(yw, rev)
        if st["merge"] is not None:
            m, tab = st["merge"]
            g = _gather(x, tab)
            gq, bq, lc = orc.layernorm_prepare(m.gamma, m.beta, m.ln_out_scale, 0)
            h = orc.layernorm(g, gq, bq, lc)
            rq = [orc.requant_prepare(float(r)) for r in m.ratio]
            x = orc.linear(h, m.w, None, np.array([r.mult for r in rq], np.int32), np.array([r.shift for r in rq], np.int8))
    return x


def test_gather_rows_matches_numpy(api):
    import torch
    rng = np.random.default_rng(0)
    src = rng.integers(-128, 128, size=(1000, 96)).astype(np.int8)
    idx = rng.integers(-1, 1000, size=(777, 4)).astype(np.int32)
    got = api.gather_rows(torch.from_numpy(src).cuda(), torch.from_numpy(idx).cuda()).cpu().numpy()
    assert (got == _gather(src, idx)).all()
    fwd, mask, rev, nW = synth.swin_window_tables(2, 10, 15, 3)
    x = rng.integers(-128, 128, size=(2 * 10 * 15, 32)).astype(np.int8)
    xw = api.gather_rows(torch.from_numpy(x).cuda(), torch.from_numpy(fwd.reshape(-1, 1)).cuda())
    back = api.gather_rows(xw, torch.from_numpy(rev.reshape(-1, 1)).cuda()).cpu().numpy()
    assert (back == x).all()                                   # partition followed by its inverse is the identity
    assert (xw.cpu().numpy()[fwd < 0] == 0).all() and (mask.reshape(-1)[fwd < 0] == synth.PAD_LABEL).all()


@pytest.mark.parametrize("name,B,stages", [
    ("two small stages", 1, [dict(dim=96, heads=3, depth=2, grid=(20, 31)), dict(dim=192, heads=6, depth=2, grid=(10, 16))]),
    ("Swin-T at 800x1216", 2, None),
])
def test_backbone_matches_the_oracle_composition(api, orc, name, B, stages):
    import torch
    from paper_2511_15369_b200 import swin
    spec = synth.make_swin(B, stages, seed=3)
    table = (0, 0, 0, 0)
    net = swin.SwinBackbone(spec, table)
    got = net(torch.from_numpy(spec.x).cuda()).cpu().numpy()
    net.check()
    want = _oracle_backbone(orc, spec, table)
    assert got.shape == want.shape and len(np.unique(want)) > 30
    bad = int((got != want).sum())
    assert bad == 0, "%d of %d elements differ" % (bad, want.size)
