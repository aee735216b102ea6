"""Whole ViT / DeiT forward pass on the GPU (patch rows, INT8 patch embedding with the position embedding on the
residual branch, class token, encoder blocks, final LayerNorm, classifier) against the oracle's composition of the
same layers: bit-exact logits and tokens."""
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


@pytest.mark.parametrize("B,C,H,W,P", [(2, 3, 224, 224, 16), (1, 3, 64, 96, 32), (3, 1, 16, 16, 16), (5, 4, 48, 32, 16)])
def test_patchify_parity(api, B, C, H, W, P):
    from oracle import compose
    img = np.random.default_rng(B + H).integers(-128, 128, size=(B, C, H, W)).astype(np.int8)
    got = api.patchify(_cu(img), P).cpu().numpy()
    assert (got == compose.patch_rows(img, P)).all()


def test_patchify_errors(api):
    import torch
    img = torch.zeros((1, 3, 32, 32), dtype=torch.int8, device="cuda")
    out = torch.zeros((4, 768), dtype=torch.int8, device="cuda")
    L = api.lib()
    assert L.iptq_patchify(img.data_ptr(), out.data_ptr(), 1, 3, 32, 32, 8, None) == api.ERR_SHAPE
    assert L.iptq_patchify(img.data_ptr(), out.data_ptr(), 1, 3, 40, 32, 16, None) == api.ERR_SHAPE
    assert L.iptq_patchify(None, out.data_ptr(), 1, 3, 32, 32, 16, None) == api.ERR_NULL
    assert L.iptq_patchify(img.data_ptr(), out.data_ptr(), 0, 3, 32, 32, 16, None) == api.OK


@pytest.mark.parametrize("name,B,depth,table", [
    ("DeiT-T", 2, 12, (0, 0, 0, 0)),
    ("DeiT-T", 3, 3, (1, 1, 1, 1)),
    ("DeiT-S", 8, 2, (0, 0, 0, 0)),
    ("DeiT-B", 1, 1, (2, 0, 1, 0)),
])
def test_vit_forward_parity(api, name, B, depth, table):
    import torch
    from oracle import compose
    from paper_2511_15369_b200 import vit
    spec = synth.make_vit(name, B, seed=7, depth=depth)
    want, want_tok = compose.vit_forward(spec, table, return_tokens=True)
    model = vit.VitModel(spec, table)
    img = _cu(spec.image)
    got = model(img).cpu().numpy()
    model.check()
    tok = model.x[depth & 1].cpu().numpy()
    assert (tok == want_tok).all(), int((tok != want_tok).sum())
    assert (got == want).all(), int((got != want).sum())
    assert len(np.unique(want)) > 20
    # the same forward pass replayed from a CUDA graph
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        model(img)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            model(img)
    model.logits_padded.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert (model.logits.cpu().numpy() == want).all()
    assert model.launches_per_forward() == 6 + 7 * depth
