"""Pins of the scale-byte layout helpers (the 128-row x 4-block atoms the block-scaled MMA reads): the C routine
`orc_sf_swizzled_offset` and the two numpy helpers `sf_swizzle` / `sf_unswizzle` every swizzled comparison goes
through.  The layout is stated in include/nvfp4.h:
    offset(r, kb) = ((r / 128) * (n_kb / 4) + kb / 4) * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4
"""
import numpy as np
import pytest

import oracle

SHAPES = [(128, 4), (128, 8), (256, 4), (384, 20), (1024, 64), (128, 320)]


def test_offsets_worked_by_hand():
    # each line: the formula of the header evaluated by hand
    assert oracle.sf_swizzled_offset(0, 0, 4) == 0
    assert oracle.sf_swizzled_offset(127, 3, 4) == 31 * 16 + 3 * 4 + 3 == 511        # last byte of the only atom
    assert oracle.sf_swizzled_offset(37, 6, 8) == 1 * 512 + 5 * 16 + 1 * 4 + 2 == 598  # atom 1; lane 5, quarter 1, block 2
    assert oracle.sf_swizzled_offset(200, 13, 20) == (1 * 5 + 3) * 512 + 8 * 16 + 2 * 4 + 1 == 4233
    assert oracle.sf_swizzled_offset(128, 0, 4) == 512                                 # the next 128 rows: next atom
    assert oracle.sf_swizzled_offset(32, 0, 4) == 4 and oracle.sf_swizzled_offset(1, 0, 4) == 16


@pytest.mark.parametrize("rows,n_kb", SHAPES)
def test_offset_map_is_a_bijection_onto_the_buffer(rows, n_kb):
    off = np.array([[oracle.sf_swizzled_offset(r, kb, n_kb) for kb in range(n_kb)] for r in range(rows)])
    assert off.min() == 0 and off.max() == rows * n_kb - 1
    assert np.unique(off).size == rows * n_kb


@pytest.mark.parametrize("rows,n_kb", SHAPES)
def test_numpy_helpers_agree_with_the_c_routine_and_invert_each_other(rows, n_kb):
    rng = np.random.default_rng(rows * 131 + n_kb)
    lin = rng.integers(0, 256, (rows, n_kb), dtype=np.uint8)
    swz = oracle.sf_swizzle(lin)
    assert swz.dtype == np.uint8 and swz.size == rows * n_kb
    # every byte sits where the C routine says
    off = np.array([[oracle.sf_swizzled_offset(r, kb, n_kb) for kb in range(n_kb)] for r in range(rows)])
    assert np.array_equal(swz.reshape(-1)[off], lin)
    assert np.array_equal(oracle.sf_unswizzle(swz, rows, n_kb), lin)
    # the other direction, from an arbitrary swizzled buffer
    buf = rng.integers(0, 256, rows * n_kb, dtype=np.uint8)
    assert np.array_equal(oracle.sf_swizzle(oracle.sf_unswizzle(buf, rows, n_kb)).reshape(-1), buf)


@pytest.mark.parametrize("rows,n_kb", SHAPES)
def test_layout_is_the_structural_statement_of_the_atom(rows, n_kb):
    """An atom holds, for 128 rows and 4 consecutive blocks, 32 units of 16 bytes: unit = row % 32, and inside a unit
    4 bytes for each of the four 32-row quarters.  Written as a reshape / transpose, without the offset formula."""
    lin = np.arange(rows * n_kb, dtype=np.int64).reshape(rows, n_kb) % 251
    lin = lin.astype(np.uint8)
    a = lin.reshape(rows // 128, 4, 32, n_kb // 4, 4)           # [row atom][quarter][row % 32][block atom][block % 4]
    structural = a.transpose(0, 3, 2, 1, 4).reshape(-1)         # [row atom][block atom][row % 32][quarter][block % 4]
    assert np.array_equal(oracle.sf_swizzle(lin).reshape(-1), structural)
