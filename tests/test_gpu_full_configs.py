"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times:
the GPU runs the whole batch through iptq_encoder_block() and the CPU oracle recomputes it; with the default
variant table every element of the batch has to match bit for bit (the last ragged items and the tail of the last
wave of tiles included), with the other tables a sample of the images (attention problems are independent, so an
image's output rows depend on that image alone).  cfg1 = DeiT-Small b64, cfg2 = ViT-Base b128 (W8A8 with alternating variant
tables, then W4A8), cfg3 = Swin-Tiny stage-1 windows with the relative-position bias."""
import copy

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


def _pick(spec, images):
    """Block spec restricted to the given images (same weights and scales)."""
    s = copy.copy(spec)
    sh = spec.shape
    s.shape = synth.BlockShape(sh.name, len(images), sh.N, sh.D, sh.H, sh.dh, sh.Dh, sh.has_bias)
    rows = np.concatenate([np.arange(i * sh.N, (i + 1) * sh.N) for i in images])
    s.x = np.ascontiguousarray(spec.x[rows])
    if spec.mask_id is not None:
        s.mask_id = np.ascontiguousarray(spec.mask_id[list(images)])
    return s, rows


@pytest.mark.parametrize("cfg,w_bits,table,gelu_bits,whole", [
    ("cfg1", 8, (0, 0, 0, 0), 16, True),
    ("cfg2", 8, (0, 0, 0, 0), 16, True),
    ("cfg2", 8, (1, 1, 1, 1), 16, False),       # the alternate candidates: Shiftmax, second-order GELU, Newton LayerNorm
    ("cfg2", 8, (2, 2, 0, 1), 14, False),       # polynomial Softmax, shift GELU
    ("cfg2", 4, (0, 0, 0, 0), 16, False),       # W4A8
    ("cfg3", 8, (0, 0, 0, 0), 16, True),
])
def test_full_size_block_matches_the_oracle(api, orc, cfg, w_bits, table, gelu_bits, whole):
    import torch
    shape = synth.CONFIGS[cfg]
    spec = synth.make_block(shape, seed=2, w_bits=w_bits, gelu_in_bits=gelu_bits)
    blk = api.EncoderBlock(spec, table)
    got = blk(torch.from_numpy(spec.x).cuda()).cpu().numpy()
    blk.ws.check()
    images = list(range(shape.B)) if whole else sorted({0, 1, shape.B // 2, shape.B - 1})
    sample, rows = _pick(spec, images)
    want = _oracle_block(orc, sample, table)
    assert len(np.unique(want)) > 30
    bad = int((got[rows] != want).sum())
    assert bad == 0, "%d of %d compared elements differ" % (bad, want.size)
    # the rest of the batch was produced too (no image left untouched): every image has a spread of values
    per_image = got.reshape(shape.B, -1)
    assert (per_image.max(axis=1) > per_image.min(axis=1)).all()
