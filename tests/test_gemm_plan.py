"""Host logic of the two-SM contraction kernel: the unit plan (no GPU).  Whatever the shape, every 128-column chunk
of every 256-row block must be computed exactly once, units must stay inside their row block and within the
accumulator memory, and the order must be the one the kernel's ring switching relies on (widest first)."""
import itertools

import numpy as np
import pytest

from paper_1810_00952_b200 import binding as B

SHAPES = [(4096, 4096, 4096), (8192, 4096, 1024), (4096, 4096, 512), (8192, 4096, 2048), (256, 37888, 4096), (4100, 4000, 4096),
          (2304, 256, 100352), (1024, 4096, 8192), (16384, 1024, 4096), (300, 40000, 64), (4096, 136, 4096), (65536, 640, 4096)]


def check_plan(M, N, K, sms):
    units = B.relay_debug_plan_units(M, N, K, sms)
    tiles_m, cpr, k_blocks = -(-M // 256), -(-N // 128), -(-K // 64)
    if units is None:
        assert tiles_m * cpr > 640          # only shapes whose list cannot fit fall back to the fixed scheme
        return None
    cover = np.zeros((tiles_m, cpr), dtype=np.int32)
    for m, c0, w in units:
        assert 0 <= m < tiles_m and 1 <= w <= 4 and c0 + w <= cpr, (m, c0, w)
        cover[m, c0:c0 + w] += 1
    assert (cover == 1).all(), (M, N, K, sms)
    widths = [w for _, _, w in units]
    assert widths == sorted(widths, reverse=True)             # widest first: a pair's units never grow in class
    if k_blocks < 32:
        assert max(widths) <= 2                                # short contractions keep the overlapped epilogue
    pairs = min(tiles_m * -(-N // 256), sms // 2)
    load = np.zeros(pairs, dtype=np.int64)
    for i, (_, _, w) in enumerate(units):
        load[i % pairs] += w
    share = -(-tiles_m * cpr // pairs)
    assert load.max() <= share + 4, (load.max(), share)        # nobody carries more than its share plus one unit
    return units


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_plan_covers_every_chunk_once(M, N, K):
    for sms in (148, 132, 2, 16):
        check_plan(M, N, K, sms)


def test_plan_over_a_grid_of_ragged_shapes():
    for M, N, K in itertools.product((256, 257, 1000, 4096, 5000), (128, 200, 384, 1000, 4096, 4104), (64, 2048, 4096)):
        check_plan(M, N, K, 148)


def test_plan_of_the_mlp_configuration():
    """4096^3 on 74 pairs: 512 chunks, 7 per pair = one unit of four and one of three (what is left at the end of a
    row block becomes a narrower unit)."""
    units = check_plan(4096, 4096, 4096, 148)
    widths = [w for _, _, w in units]
    assert len(units) == 148 and widths.count(4) == 74 and widths.count(3) == 68 and widths.count(2) == 6


def test_bad_arguments_are_refused():
    with pytest.raises(ValueError):
        B.relay_debug_plan_units(0, 128, 64, 148)
    with pytest.raises(ValueError):
        B.relay_debug_plan_units(4096, 4096, 4096, 148, max_units=8)
