"""Host logic of the GEMM launch plan (no GPU): the partition `zq_w4a8_linear_plan` reports is replayed in
Python from the rules stated in include/zqfp.h and must cover every (output tile, K block) unit exactly once,
map launch positions to tiles one-to-one, and leave enough partial-sum scratch for the tiles that CTAs share."""
import itertools

import numpy as np
import pytest

from paper_2307_09782_b200 import binding

SHAPES = [(1, 768, 768), (8192, 7296, 28672), (1120, 15488, 512), (8, 28672, 7168), (16, 7168, 28672), (17, 4096, 4096), (32, 28672, 7168), (64, 129, 1024),
          (100, 384, 512), (128, 28672, 7168), (128, 7168, 28672), (130, 384, 512), (192, 256, 512), (200, 300, 512),
          (300, 384, 512), (500, 640, 2048), (512, 28672, 7168), (512, 7168, 28672), (700, 1000, 1024),
          (1000, 15360, 512), (1120, 15360, 9216), (2048, 28672, 7168), (2048, 7168, 28672), (2048, 4096, 11008),
          (4096, 6656, 17920), (8192, 28672, 7168), (8192, 7168, 28672), (5000, 128, 128), (33, 128, 128)]


def raster(pos, m_tiles, n_tiles, m_group):
    if m_group <= 1:
        return pos
    per_group = m_group * n_tiles
    g, within = divmod(pos, per_group)
    gm = min(m_group, m_tiles - g * m_group)
    return (g * m_group + within % gm) * n_tiles + within // gm


def pair_raster(pp, m_tiles, n_pairs, m_group):
    mg = max(1, m_group)
    per_group = mg * n_pairs
    g, within = divmod(pp, per_group)
    gm = min(mg, m_tiles - g * mg)
    return g * mg + within % gm, within // gm


def units_of_cta(pl, c, kblocks):
    """(position, K block) units of CTA c, in order."""
    tiles = pl["m_tiles"] * pl["n_tiles"]
    out = []

    def dealt(first_unit):
        start = first_unit + c * pl["base"] + min(c, pl["rem"])
        end = first_unit + (c + 1) * pl["base"] + min(c + 1, pl["rem"])
        return [(u // kblocks, u % kblocks) for u in range(start, end)]

    if pl["pair"]:
        # CTAs 2c and 2c + 1 are pair c: they share the token tile of each of the pair's positions and CTA 2c + h
        # takes the channel tile 2 * n_pair + h.  Positions, tail_pos0 and base / rem count pair positions and pairs.
        # Units are reported by tile index here, not by launch position.
        pairs, (pair, half) = pl["ctas"] // 2, divmod(c, 2)

        def dealt_pair(first_unit):
            start = first_unit + pair * pl["base"] + min(pair, pl["rem"])
            end = first_unit + (pair + 1) * pl["base"] + min(pair + 1, pl["rem"])
            return [(u // kblocks, u % kblocks) for u in range(start, end)]

        if pl["stream"]:
            us = dealt_pair(0)
        else:
            us = [(pp, kb) for pp in range(pair, pl["tail_pos0"], pairs) for kb in range(kblocks)]
            us += dealt_pair(pl["tail_pos0"] * kblocks)
        for pp, kb in us:
            m_tile, n_pair = pair_raster(pp, pl["m_tiles"], pl["n_tiles"] // 2, pl["m_group"])
            out.append((m_tile * pl["n_tiles"] + 2 * n_pair + half, kb))
        return out
    if pl["stream"]:
        return dealt(0)
    if pl["persist"]:
        for pos in range(c, pl["tail_pos0"], pl["ctas"]):
            out += [(pos, kb) for kb in range(kblocks)]
        return out + dealt(pl["tail_pos0"] * kblocks)
    z, pos = divmod(c, tiles)
    k0 = z * pl["kb_per_split"]
    return [(pos, kb) for kb in range(k0, min(k0 + pl["kb_per_split"], kblocks))]


@pytest.mark.parametrize("layout,mode", [("cast", "M2"), ("cast", "none"), ("mx", "M1")])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_plan_covers_every_unit_once(M, N, K, layout, mode):
    pl = binding.linear_plan(M, N, K, mode, layout)
    bm, m_tiles, n_tiles, ctas = pl["bm"], pl["m_tiles"], pl["n_tiles"], pl["ctas"]
    kblocks = K // 128
    tiles = m_tiles * n_tiles
    assert m_tiles == -(-M // bm) and n_tiles == -(-N // 128) and ctas >= 1
    assert not (pl["stream"] and pl["persist"])
    # launch order -> tile is a permutation
    perm = [raster(p, m_tiles, n_tiles, pl["m_group"]) for p in range(tiles)]
    assert sorted(perm) == list(range(tiles))
    # exact cover; per CTA the units are contiguous runs per tile, so a CTA leaves at most two partial tiles
    seen = np.zeros((tiles, kblocks), dtype=np.int32)
    sharers = np.zeros(tiles, dtype=np.int32)
    max_partial_tiles = 0
    for c in range(ctas):
        us = units_of_cta(pl, c, kblocks)
        partial = 0
        for pos, grp in itertools.groupby(us, key=lambda u: u[0]):
            kbs = [kb for _, kb in grp]
            assert kbs == list(range(kbs[0], kbs[0] + len(kbs)))
            for kb in kbs:
                seen[pos, kb] += 1
            sharers[pos] += 1
            partial += len(kbs) < kblocks
        max_partial_tiles = max(max_partial_tiles, partial)
    assert np.all(seen == 1), (pl, np.argwhere(seen != 1)[:4])
    # scratch: dealt ranges leave at most two partial tiles per CTA (slots 2c, 2c + 1); split K one per CTA
    shared = sharers > 1
    if shared.any():
        assert tiles <= 16384, "shared tiles are counted in the workspace's tile counters"
        if pl["pair"]:
            assert max_partial_tiles <= 2   # shared tiles are handed over by flags into an FP32 y: no scratch
        elif pl["stream"] or pl["persist"]:
            assert max_partial_tiles <= 2
            assert pl["partial_floats"] >= 2 * ctas * bm * 128
        else:
            assert pl["partial_floats"] >= tiles * pl["splits"] * bm * 128
    ws = binding.linear_workspace_bytes(M, N, K, 8)
    assert ws >= 256 + 4 * 16384 + 4 * pl["partial_floats"]


def test_plan_tile_choices_of_the_block_scaled_kernel():
    # one row of tiles up to 256 tokens, then 192 / 224 (two accumulators) or 256 (long rows, many tiles)
    assert [binding.linear_plan(M, 28672, 7168, "M2", "mx")["bm"] for M in (1, 16, 17, 64, 100, 192, 256)] == \
        [16, 16, 32, 64, 128, 192, 256]
    assert binding.linear_plan(512, 28672 + 128, 7168, "M2", "mx")["bm"] == 192   # odd channel-tile count: single CTAs
    assert binding.linear_plan(8192, 28672, 7168, "M2", "mx")["bm"] == 224
    # many tokens, an even number of channel tiles: CTA pairs on whole tiles, the tile width with the fewest
    # rounds x width (37 x 28 pair positions of 224 tokens are 14 whole rounds of 74 pairs)
    p = binding.linear_plan(8192, 7168, 28672, "M2", "mx")
    if p["sms"] == 148:
        assert p["pair"] == 1 and p["persist"] == 1 and p["bm"] == 224 and p["ctas"] == 148 and p["partial_floats"] == 0
        assert p["tail_pos0"] == 37 * 28                      # 14 whole rounds, nothing left to deal out
        p = binding.linear_plan(4096, 6656, 17920, "M2", "mx")     # 20 x 26 positions of 208 tokens: 7 rounds, 2 positions dealt out
        assert p["pair"] == 1 and p["persist"] == 1 and p["bm"] == 208 and p["tail_pos0"] == 7 * 74
        assert p["base"] * 74 + p["rem"] == 2 * 140
        p = binding.linear_plan(2048, 7168, 28672, "M2", "mx")     # 10 x 28 positions: fewer than four rounds, all dealt out
        assert p["pair"] == 1 and p["stream"] == 1 and p["bm"] == 208 and p["base"] * 74 + p["rem"] == 280 * 224
        p = binding.linear_plan(512, 7168, 28672, "M2", "mx")      # three tiles of 176 tokens instead of 192
        assert p["pair"] == 1 and p["stream"] == 1 and p["bm"] == 176 and p["base"] * 74 + p["rem"] == 84 * 224
    # an odd number of channel tiles: single CTAs, whole rounds of whole tiles and a dealt-out last round
    p = binding.linear_plan(8192, 7168 + 128, 28672, "M2", "mx")
    assert p["pair"] == 0 and p["persist"] == 1 and p["bm"] == 256
    assert p["tail_pos0"] == (32 * 57) // p["ctas"] * p["ctas"]   # 12 whole rounds
    assert binding.linear_plan(8192, 28672, 7168, "none", "mx")["pair"] == 0
    # unconstrained scales: the running sums of a tile live in registers, so its token tiles stop at 128
    assert [binding.linear_plan(M, 4096, 4096, "none", "mx")["bm"] for M in (16, 100, 300, 2048)] == [16, 128, 128, 128]
    with pytest.raises(binding.ZqError):
        binding.linear_plan(16, 128, 256, "none", "mx_fp8")
