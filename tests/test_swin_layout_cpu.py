"""Host-side layout tables of the Swin-shaped backbone against plain numpy reshapes, rolls and slices."""
import numpy as np
import pytest

from paper_2511_15369_b200 import synth


@pytest.mark.parametrize("B,Hh,Ww,shift", [(1, 14, 21, 0), (2, 10, 15, 3), (1, 25, 38, 3), (2, 7, 7, 0)])
def test_window_tables_match_pad_roll_reshape(B, Hh, Ww, shift):
    w = 7
    fwd, mask, rev, nW = synth.swin_window_tables(B, Hh, Ww, shift, w)
    Hp, Wp = -(-Hh // w) * w, -(-Ww // w) * w
    assert nW == (Hp // w) * (Wp // w) and fwd.shape == (B * nW * w * w,) and mask.shape == (B * nW, w * w)
    tok = np.arange(1, B * Hh * Ww + 1).reshape(B, Hh, Ww)                 # token number + 1, 0 = padding
    pad = np.zeros((B, Hp, Wp), dtype=tok.dtype)
    pad[:, :Hh, :Ww] = tok
    rolled = np.roll(pad, (-shift, -shift), axis=(1, 2))
    win = rolled.reshape(B, Hp // w, w, Wp // w, w).transpose(0, 1, 3, 2, 4).reshape(-1)
    assert (win - 1 == fwd).all()
    # the inverse table brings every token back
    assert (fwd[rev] == np.arange(B * Hh * Ww)).all()
    # labels: padding carries its own label; without a shift all real tokens share one label
    assert ((mask.reshape(-1) == synth.PAD_LABEL) == (fwd < 0)).all()
    if shift == 0:
        assert set(np.unique(mask)) <= {0, synth.PAD_LABEL}
    else:
        # two real tokens of a window share a label iff they were neighbours before the roll (no wrap between them)
        lab = mask.reshape(B, nW, w * w)[0]
        src = fwd.reshape(B, nW, w * w)[0]
        for wi in (0, nW - 1, nW // 2):
            ok = src[wi] >= 0
            i, j = src[wi][ok] // Ww, src[wi][ok] % Ww
            same = lab[wi][ok][:, None] == lab[wi][ok][None, :]
            near = (np.abs(i[:, None] - i[None, :]) < w) & (np.abs(j[:, None] - j[None, :]) < w)
            assert (same == near).all()


def test_merge_table_matches_strided_slices():
    B, Hh, Ww, C = 2, 6, 10, 3
    x = np.arange(B * Hh * Ww * C).reshape(B, Hh, Ww, C)
    want = np.concatenate([x[:, 0::2, 0::2], x[:, 1::2, 0::2], x[:, 0::2, 1::2], x[:, 1::2, 1::2]], axis=-1).reshape(-1, 4 * C)
    tab = synth.swin_merge_table(B, Hh, Ww)
    got = np.concatenate([x.reshape(-1, C)[tab[:, p]] for p in range(4)], axis=1)
    assert (got == want).all()
    assert (synth.swin_merge_table(1, 5, 4)[:, 1].reshape(3, 2)[2] == -1).all()      # odd grid: no token below the last row
