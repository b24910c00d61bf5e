"""The device routine for stochastic rounding (Section 4.4) against the oracle's scalar rule, value by value.

The kernels round with the hardware conversion instruction fed a pre-biased magnitude and a crafted random word; this
sweep shows that it takes the oracle's decision for EVERY one of the 256 draws on a dense set of binary32 inputs:
zeros of both signs, denormals, every grid point and binade edge with its neighbours, every decision threshold
lo + step * (u + 0.5) / 256 with its neighbours, saturating magnitudes, and a uniform sweep of [-6.5, 6.5].
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_25149_b200 import binding as B

pytestmark = pytest.mark.gpu
GRID = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def _neighbours(x, k):
    out, lo, hi = [np.float32(x)], np.float32(x), np.float32(x)
    for _ in range(k):
        lo, hi = np.nextafter(lo, np.float32(-10)), np.nextafter(hi, np.float32(10))
        out += [lo, hi]
    return out


def sweep_values():
    rng = np.random.default_rng(20250925)
    vals = [np.float32(0.0), np.float32(-0.0)]
    for g in GRID[1:]:
        vals += _neighbours(g, 48)
    for i in range(7):                       # every decision threshold of every cell, and its float neighbours
        lo, step = GRID[i], GRID[i + 1] - GRID[i]
        for u in range(256):
            vals += _neighbours(lo + step * (u + 0.5) / 256.0, 2)
    vals += list(np.linspace(-6.5, 6.5, 40001).astype(np.float32))
    vals += list((rng.random(40000) * 6.5).astype(np.float32))
    vals += list((rng.random(10000) * 1.0).astype(np.float32))
    vals += list((rng.random(10000) * 2.0 ** -6).astype(np.float32))
    vals += [np.float32(x) for x in (1e-38, 1e-40, 1.4e-45, 2.0 ** -126, 2.0 ** -20, 6.0000005, 6.5, 7.0, 448.0, 3e38)]
    v = np.array(vals, dtype=np.float32)
    return np.concatenate([v, -v])


def test_every_draw_on_a_dense_sweep_matches_the_oracle():
    v = sweep_values()
    vd = torch.from_numpy(v).cuda()
    bad = 0
    for u in range(256):
        draws = np.full(v.size, u, dtype=np.uint8)
        got = B.nvfp4_e2m1_sr(vd, torch.from_numpy(draws).cuda()).cpu().numpy()
        want = oracle.e2m1_encode_sr_many(v, draws)
        diff = np.flatnonzero(got != want)
        if diff.size:
            i = diff[0]
            raise AssertionError(f"draw {u}: {diff.size} values differ, e.g. v = {v[i]!r} (bits {v[i:i+1].view(np.uint32)[0]:#x}) "
                                 f"-> {got[i]} instead of {want[i]}")
        bad += diff.size
    assert bad == 0


def test_random_values_with_random_draws():
    rng = np.random.default_rng(7)
    v = (rng.standard_normal(1 << 20) * 2.5).astype(np.float32)
    u = rng.integers(0, 256, v.size, dtype=np.uint8)
    got = B.nvfp4_e2m1_sr(torch.from_numpy(v).cuda(), torch.from_numpy(u).cuda()).cpu().numpy()
    assert np.array_equal(got, oracle.e2m1_encode_sr_many(v, u))
