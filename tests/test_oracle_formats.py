"""Pins for the oracle's number formats, rounding rules and random source (CPU only)."""
import ctypes
import os
import subprocess

import numpy as np
import pytest
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))
GOLD = os.path.join(HERE, "golden")


def _golden_lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


@pytest.fixture(scope="module")
def nv_host():
    """NVIDIA's host-side conversion routines (cuda_fp4.h / cuda_fp8.h), test-only cross-check."""
    inc = "/usr/local/cuda/include"
    if not os.path.exists(os.path.join(inc, "cuda_fp4.h")):
        pytest.skip("CUDA toolkit headers not present")
    so = os.path.join(HERE, "libnv_host_cvt.so")
    src = os.path.join(HERE, "nv_host_cvt.cpp")
    if not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
        tmp = f"{so}.{os.getpid()}.tmp"
        subprocess.run(["g++", "-O1", "-fPIC", "-shared", f"-I{inc}", "-o", tmp, src], check=True)
        os.replace(tmp, so)
    L = ctypes.CDLL(so)
    for fn in (L.nv_host_e2m1_rne, L.nv_host_e4m3_satfinite):
        fn.restype, fn.argtypes = ctypes.c_uint8, [ctypes.c_float]
    return L


# ------------------------------------------------------------------ E2M1 ----
def test_e2m1_value_set_is_the_papers():
    mags = [float(v) for v in _golden_lines("e2m1_values.txt")]
    assert [oracle.e2m1_decode(c) for c in range(8)] == mags
    assert [oracle.e2m1_decode(c | 8) for c in range(8)] == [-m for m in mags]
    assert max(mags) == 6.0 and min(m for m in mags if m > 0) == 0.5


def test_e2m1_rne_ties_and_saturation():
    # every midpoint of the grid goes to the neighbour with mantissa bit 0
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for v, want in ties.items():
        assert oracle.e2m1_decode(oracle.e2m1_encode_rne(v)) == want
        assert oracle.e2m1_decode(oracle.e2m1_encode_rne(-v)) == -want
        # one float step away from the tie the nearer neighbour wins
        up, dn = np.nextafter(np.float32(v), np.float32(9)), np.nextafter(np.float32(v), np.float32(0))
        assert oracle.e2m1_decode(oracle.e2m1_encode_rne(up)) > oracle.e2m1_decode(oracle.e2m1_encode_rne(dn))
    for v in (6.0, 6.5, 1e9, float("inf")):
        assert oracle.e2m1_encode_rne(v) == 7 and oracle.e2m1_encode_rne(-v) == 15
    assert oracle.e2m1_encode_rne(0.0) == 0 and oracle.e2m1_encode_rne(-0.0) == 8
    assert oracle.e2m1_encode_rne(-0.1) == 8  # sign survives a magnitude that rounds to zero


def test_e2m1_rne_matches_toolkit_host_routine(nv_host):
    rng = np.random.default_rng(7)
    xs = np.concatenate([np.linspace(-8, 8, 6401, dtype=np.float32),
                         rng.standard_normal(4000).astype(np.float32) * 3,
                         np.array([0.0, 1e-30, 5.0, 2.5, 1e30], dtype=np.float32)])
    for x in xs:
        got, want = oracle.e2m1_encode_rne(float(x)), nv_host.nv_host_e2m1_rne(float(x))
        if x == 0 or abs(oracle.e2m1_decode(got)) == 0:
            assert (got & 7) == (want & 7)  # the library drops the sign of a zero result or not: magnitude only
        else:
            assert got == want, x


def test_e2m1_rne_is_nearest_by_error_bound():
    # |v - q(v)| <= half the local grid step: 0.25 below 2, 0.5 on [2,4), 1 on [4,6]
    for v in np.linspace(0, 6, 2401):
        q = oracle.e2m1_decode(oracle.e2m1_encode_rne(float(v)))
        bound = 0.25 if v < 2 else (0.5 if v < 4 else 1.0)
        assert abs(np.float32(v) - q) <= bound


# ------------------------------------------------------------------ E4M3 ----
def test_e4m3_decode_matches_torch_for_all_bytes():
    b = torch.arange(256, dtype=torch.int16).to(torch.uint8)
    ref = b.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for i in range(256):
        mine = oracle.e4m3_decode(i)
        if np.isnan(ref[i]):
            assert np.isnan(mine)
        else:
            assert mine == ref[i], i
    assert oracle.e4m3_decode(0x7E) == 448.0 and oracle.e4m3_decode(0x38) == 1.0
    assert oracle.e4m3_decode(0x01) == 2.0 ** -9
    finite_nonneg = [oracle.e4m3_decode(i) for i in range(0x7F)]
    assert len(set(finite_nonneg)) == 127 and max(finite_nonneg) == 448.0
    assert all(x < y for x, y in zip(finite_nonneg, finite_nonneg[1:]))  # byte order == value order


def test_e4m3_encode_matches_torch_and_toolkit(nv_host):
    rng = np.random.default_rng(11)
    xs = np.concatenate([
        np.exp(rng.uniform(np.log(2.0 ** -12), np.log(448.0), 6000)).astype(np.float32),
        np.array([0.0, 2.0 ** -10, 2.0 ** -10 * 1.0001, 2.0 ** -9 * 1.5, 447.9, 448.0, 464.0], np.float32)])
    # every midpoint between consecutive E4M3 values, and its float neighbours
    vals = np.array([oracle.e4m3_decode(i) for i in range(0x7F)], dtype=np.float64)
    mids = ((vals[1:] + vals[:-1]) / 2).astype(np.float32)
    xs = np.concatenate([xs, mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9))])
    t = torch.from_numpy(xs).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for x, tb in zip(xs, t):
        got = oracle.e4m3_encode_rne(float(x))
        assert got == nv_host.nv_host_e4m3_satfinite(float(x)), x
        assert got == tb, x
    # saturation (torch's cast is not saturating, so only the toolkit routine is compared here)
    for x in (480.0, 1e4, 3e38):
        assert oracle.e4m3_encode_rne(x) == 0x7E == nv_host.nv_host_e4m3_satfinite(x)


# ---------------------------------------------------------------- Philox ----
def test_philox_known_answers():
    for ln in _golden_lines("philox4x32_10_kat.txt"):
        w = [int(t, 16) for t in ln.split()]
        assert oracle.philox4x32_10(w[0:4], w[4:6]).tolist() == w[6:10]


def test_sr_draw_indexing():
    # seed 0, offset 0, group 0: output word 0 is 0x6627e8d5, bytes taken little-endian
    assert [oracle.sr_draw(0, 0, e) for e in range(4)] == [0xD5, 0xE8, 0x27, 0x66]
    out = oracle.philox4x32_10([5, 0, 9, 0], [3, 0])
    raw = out.astype("<u4").tobytes()
    assert [oracle.sr_draw(3, 9, 5 * 16 + i) for i in range(16)] == list(raw)
    # 64-bit group index and 64-bit seed / offset reach the high counter / key words
    e = (1 << 40) + 7
    out = oracle.philox4x32_10([(e >> 4) & 0xFFFFFFFF, (e >> 4) >> 32, 2, 1], [4, 6])
    assert oracle.sr_draw((6 << 32) | 4, (1 << 32) | 2, e) == out.astype("<u4").tobytes()[7]


# --------------------------------------------------- stochastic rounding ----
def test_sr_rule_on_the_first_draws():
    # v = 2.25 sits a quarter of the way from 2 to 3: 256*frac = 64; draws D5 E8 27 66
    got = [oracle.e2m1_decode(oracle.e2m1_encode_sr(2.25, oracle.sr_draw(0, 0, e))) for e in range(4)]
    assert got == [2.0, 2.0, 3.0, 2.0]


def test_sr_neighbours_grid_points_and_symmetry():
    grid = [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    for g in grid:  # representable values never move
        for u in (0, 1, 127, 128, 255):
            assert oracle.e2m1_decode(oracle.e2m1_encode_sr(g, u)) == g
            assert oracle.e2m1_decode(oracle.e2m1_encode_sr(-g, u)) == -g or g == 0
    rng = np.random.default_rng(3)
    for v in rng.uniform(0, 6.5, 300).astype(np.float32):
        lo = max(g for g in grid if g <= min(v, 6))
        hi = min([g for g in grid if g > v] or [6])
        ups = 0
        for u in range(256):
            q = oracle.e2m1_decode(oracle.e2m1_encode_sr(float(v), u))
            assert q in (lo, hi)
            ups += q == hi and hi != lo
            assert oracle.e2m1_decode(oracle.e2m1_encode_sr(-float(v), u)) == -q
        if v < 6:
            frac = (float(v) - lo) / (hi - lo)
            assert abs(ups / 256 - frac) <= 1 / 512 + 1e-12  # P(up) within 1/512 of the position
    # monotone in the draw: a smaller u can only round further up
    for v in (0.3, 1.1, 2.9, 5.5):
        qs = [oracle.e2m1_decode(oracle.e2m1_encode_sr(v, u)) for u in range(256)]
        assert all(a >= b for a, b in zip(qs, qs[1:]))
    assert oracle.e2m1_encode_sr(7.0, 255) == 7 and oracle.e2m1_encode_sr(-1e9, 0) == 15
    assert oracle.e2m1_encode_sr(-0.0, 0) == 8


def test_sr_is_unbiased_over_seeds():
    # mean over S seeds of the decoded value approaches x: |mean - x| <= step*(1/512 + 2/sqrt(S))
    S = 4096
    rng = np.random.default_rng(5)
    for v in rng.uniform(0.05, 5.9, 24).astype(np.float32):
        acc = 0.0
        for seed in range(S):
            acc += oracle.e2m1_decode(oracle.e2m1_encode_sr(float(v), oracle.sr_draw(seed, 0, 37)))
        step = 0.5 if v < 2 else (1.0 if v < 4 else 2.0)
        assert abs(acc / S - float(v)) <= step * (1 / 512 + 2 / np.sqrt(S)), v
