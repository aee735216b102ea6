"""Host-side tiling plan of the INT8 linear layer (`iptq_linear_plan`): no GPU is touched when the SM count is given.
The plan must fit the SM for every admissible shape, and the choices documented for it must hold: the widest tile
that leaves a ring of three stages (or one per block of K plus one), CTA pairs only for long reductions with enough
tiles, an even grid for pairs, never more CTAs than SMs."""
import itertools

import pytest

from paper_2511_15369_b200 import api

SMEM_LIMIT = 227 * 1024


def plan(M, N, K, **kw):
    return api.linear_plan(M, N, K, sm_count=kw.pop("sm_count", 148), **kw)


@pytest.mark.parametrize("residual,table", [(False, False), (True, False), (False, True)])
def test_every_admissible_shape_gets_a_plan_that_fits_the_sm(residual, table):
    Ms = [1, 5, 64, 65, 128, 192, 193, 197, 256, 257, 1000, 12608, 25216, 200704]
    Ns = [16, 96, 144, 288, 384, 768, 1008, 1152, 2304, 3072]
    Ks = [16, 96, 144, 272, 384, 768, 1536, 1552, 3072, 4096]
    for M, N, K in itertools.product(Ms, Ns, Ks):
        p = plan(M, N, K, residual=residual, gelu_table=table)
        kblocks = (K + 127) // 128
        assert p.tile_tokens in (64, 128, 192, 256)
        assert 1024 < p.smem_bytes <= SMEM_LIMIT, (M, N, K, p.smem_bytes)
        assert 2 <= p.stages <= 8
        assert p.staging_buffers in (1, 2)
        assert p.stages >= min(3, kblocks + 1) or p.cta_pairs, (M, N, K, p.stages)
        assert p.channel_tiles == (N + 127) // 128
        assert p.token_tiles == (M + p.tile_tokens - 1) // p.tile_tokens
        assert 1 <= p.grid <= 148
        if p.cta_pairs:
            assert p.tile_tokens == 256 and p.grid % 2 == 0 and kblocks >= 6 and p.channel_tiles >= 2
            assert ((p.channel_tiles + 1) // 2) * p.token_tiles >= 3 * 74  # three rounds of tiles per pair of SMs
        else:
            assert p.grid == min(148, p.channel_tiles * p.token_tiles)
        if M <= 64:
            assert p.tile_tokens == 64          # a wider tile would be mostly padding


def test_small_batches_take_narrow_tiles():
    # less than one round of 256-token tiles: the narrowest tile that still fits one round of 148 SMs, else 128
    assert plan(197, 576, 192).tile_tokens == 64 and plan(197, 192, 768, residual=True).tile_tokens == 64
    assert plan(1576, 1152, 384).tile_tokens == 128                      # 9 x 25 tiles of 64 tokens are too many
    assert plan(1576, 384, 1536, residual=True).tile_tokens == 64        # 3 x 25 fit
    assert plan(1576, 768, 3072, residual=True).tile_tokens == 128
    assert plan(1576, 2304, 768).tile_tokens == 128 and plan(1576, 2304, 768).cta_pairs == 0
    # one round or more at 256 tokens: unchanged
    assert plan(12608, 384, 384, residual=True).tile_tokens == 256


def test_the_configurations_of_the_benchmark():
    # short reductions have room for two staging buffers per epilogue warp, the long ones of ViT-Base keep their ring
    assert plan(200704, 96, 96, residual=True).staging_buffers == 2 and plan(200704, 288, 96).staging_buffers == 2
    assert plan(25216, 768, 3072, residual=True).staging_buffers == 1 and plan(25216, 2304, 768).staging_buffers == 1
    # ViT-Base batch 128: all four linear layers on CTA pairs
    assert (plan(25216, 2304, 768).tile_tokens, plan(25216, 2304, 768).cta_pairs) == (256, 1)
    assert plan(25216, 768, 768, residual=True).cta_pairs == 1
    assert plan(25216, 3072, 768, gelu_table=True).cta_pairs == 1
    # DeiT-Small batch 64: three blocks of K, single CTAs
    assert plan(12608, 1152, 384).cta_pairs == 0
    fc2 = plan(25216, 768, 3072, residual=True)
    assert (fc2.tile_tokens, fc2.cta_pairs, fc2.grid) == (256, 1, 148)
    # DeiT-Small batch 64: FC2 has 12 blocks of K but only two rounds of wide tiles: half-width tiles, no pairs
    fc2s = plan(12608, 384, 1536, residual=True)
    assert (fc2s.tile_tokens, fc2s.cta_pairs) == (128, 0)
    # a small device gets a smaller grid, and no pairs on a single SM
    assert plan(25216, 768, 3072, residual=True, sm_count=1).cta_pairs == 0
    assert plan(25216, 768, 3072, residual=True, sm_count=20).grid == 20


def test_shapes_the_layer_rejects_are_rejected_by_the_plan():
    for M, N, K in [(0, 128, 128), (128, 8, 128), (128, 128, 8), (128, 130, 128), (128, 128, 4112), (128, 128, 100)]:
        with pytest.raises(api.IptqError):
            plan(M, N, K)
