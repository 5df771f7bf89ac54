"""Host logic of the input-projection kernel's tiling, checked without a GPU.

The kernel numbers its 128-row x bn-column output tiles panel-major and gives each block a contiguous range of
them: either equal ranges over all tiles, or (m_ranges > 0) one panel per block and one of m_ranges ranges of the
panel's m-tiles.  Whatever the launcher chooses, every tile must belong to exactly one block, no block may be
asked for more tiles than the plan states, the grid must fit the device and the panel plus the x ring must fit
in shared memory.  The test replays the range computation of the kernel over the shapes of the five benchmark
configurations, ragged shapes and a sweep of device sizes.
"""
import itertools

import pytest

from paper_2101_05453_b200.binding import QlstmError, projection_plan

BM, BK = 128, 128


def block_ranges(rows, n, pl):
    """[t_begin, t_end) per block, as the kernel computes them from its launch parameters."""
    tiles_m, tiles_n = -(-rows // BM), -(-n // pl["bn"])
    n_tiles = tiles_m * tiles_n
    out = []
    for b in range(pl["grid"]):
        if pl["m_ranges"] > 0:
            n_tile, r = b % tiles_n, b // tiles_n
            per = -(-tiles_m // pl["m_ranges"])
            mb = min(r * per, tiles_m)
            me = min(mb + per, tiles_m)
            out.append((n_tile * tiles_m + mb, n_tile * tiles_m + me))
        else:
            per = -(-n_tiles // pl["grid"])
            tb = b * per
            out.append((tb, min(tb + per, n_tiles)))
    return out, n_tiles, tiles_m


SHAPES = [
    (20, 128, 16), (800, 1024, 80), (800, 1024, 256), (6400, 8192, 512), (32000, 3072, 640), (32000, 3072, 1024),
    (300, 8192, 640), (2400, 8192, 640), (19200, 8192, 640), (76800, 8192, 640),
    (1, 8, 16), (129, 40, 48), (350, 800, 96), (5000, 1000, 1040), (77, 8200, 2048), (100000, 24, 5120),
]


@pytest.mark.parametrize("rows,n,k", SHAPES)
@pytest.mark.parametrize("sm_count", [1, 7, 132, 148])
@pytest.mark.parametrize("max_rows_factor", [1, 3, 400], ids=["as-created", "third", "tiny-part"])
def test_every_tile_belongs_to_exactly_one_block(rows, n, k, sm_count, max_rows_factor):
    # the panel width is fixed when the handle is created (for max_rows); launches may be much smaller
    pl = projection_plan(rows, n, k, sm_count=sm_count, max_rows=rows * max_rows_factor)
    assert 32 <= pl["bn"] <= 256 and pl["bn"] % 32 == 0
    assert 2 <= pl["stages"] <= 6
    kb = -(-k // BK)
    assert kb * BK * pl["bn"] <= 160 * 1024
    assert 1024 + kb * BK * pl["bn"] + pl["stages"] * BM * BK + 16 * 64 * 4 <= 232448
    assert 1 <= pl["grid"] <= sm_count
    ranges, n_tiles, tiles_m = block_ranges(rows, n, pl)
    seen = [0] * n_tiles
    for tb, te in ranges:
        assert te - tb <= pl["per_cta"]
        if pl["m_ranges"] > 0:                            # one panel per block, and no block left without work
            assert te > tb and tb // tiles_m == (te - 1) // tiles_m
        for t in range(tb, te):
            seen[t] += 1
    assert seen == [1] * n_tiles


def test_one_panel_per_block_never_costs_more_tiles_than_equal_ranges():
    for rows, n, k in SHAPES:
        pl = projection_plan(rows, n, k)
        n_tiles = -(-rows // BM) * -(-n // pl["bn"])
        assert pl["per_cta"] <= -(-n_tiles // min(n_tiles, 148))


def test_headline_shape_fills_the_device_with_one_panel_per_block():
    # 8192 gate rows in 37 panels of 224 x 4 ranges of 150 m-tiles = 148 blocks, a whole x tile (5 k-blocks) in the ring
    pl = projection_plan(76800, 8192, 640)
    assert pl == {"bn": 224, "stages": 5, "per_cta": 150, "m_ranges": 4, "grid": 148}


def test_arguments_are_checked():
    for bad in [(0, 8, 16), (1, 0, 16), (1, 8, 0)]:
        with pytest.raises(QlstmError):
            projection_plan(*bad)
    with pytest.raises(QlstmError):
        projection_plan(200, 8, 16, max_rows=100)         # more rows than the handle was created for
    with pytest.raises(QlstmError):
        projection_plan(1000, 1024, 8192)               # a 32-row panel of 8192 columns does not fit
