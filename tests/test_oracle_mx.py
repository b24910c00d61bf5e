"""Pins for the MXFP4 part of the CPU oracle (the paper's comparison format: Section 2, Section 5, Appendix B.4):
the worked example the paper prints, closed forms of the power-of-two scale, invariants that follow from rounding the
decode scale up, the order-32 Hadamard structure, and the block / copy layout."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_25149_b200 import synth


def _bits(values):
    return synth.bits(torch.tensor(values, dtype=torch.float32).to(torch.bfloat16).reshape(1, -1))


def test_ue8m0_is_a_power_of_two_per_byte():
    for b in range(255):
        assert oracle.ue8m0_decode(b) == math.ldexp(1.0, b - 127)
    assert oracle.ue8m0_decode(127) == 1.0
    # encode scale is the exact reciprocal
    for b in range(255):
        assert float(oracle.mx_block_encode_scale(b)) * oracle.ue8m0_decode(b) == 1.0


def test_papers_worked_example_amax_three_plus_delta():
    """Appendix B.4: a block with amax = 3 + delta has decode scale 0.5 + delta/6, rounded up to 1; the amax
    element then quantizes to 3, so the samples 4 and 6 are never used by that block."""
    amax = 3.015625  # 3 + 2^-6, exact in bf16
    block = [amax, -2.0, 1.0, 0.5] + [0.0] * 28
    q = oracle.quantize_mx(_bits(block))
    assert q.scales[0, 0] == 127 and oracle.ue8m0_decode(127) == 1.0
    codes = [(q.codes[0, i // 2] >> (4 * (i & 1))) & 15 for i in range(4)]
    assert [oracle.e2m1_decode(c) for c in codes] == [3.0, -2.0, 1.0, 0.5]
    # without the delta the same block uses the full range: scale 0.5, amax -> 6
    block[0] = 3.0
    q = oracle.quantize_mx(_bits(block))
    assert q.scales[0, 0] == 126
    assert oracle.e2m1_decode(q.codes[0, 0] & 15) == 6.0


def test_scale_is_the_smallest_power_of_two_that_avoids_saturation():
    rng = np.random.default_rng(0)
    amaxes = np.concatenate([np.float32(2.0) ** rng.integers(-100, 100, 2000) * rng.uniform(1, 2, 2000).astype(np.float32),
                             np.float32([6.0, 3.0, 1.5, 0.75, 12.0, 6.0000005, 5.9999995])])
    for a in amaxes.astype(np.float32):
        b = oracle.mx_block_scale_byte(a)
        e = b - 127
        assert 6.0 * 2.0 ** e >= float(a), "scaled block would exceed 6"
        assert 6.0 * 2.0 ** (e - 1) < float(a), "a smaller power of two would have sufficed"
        # closed form from the binary representation: amax = m * 2^E with m in [1, 2): e = E - 2 if m <= 1.5 else E - 1
        m, E = math.frexp(float(a))  # m in [0.5, 1)
        m, E = 2 * m, E - 1
        assert e == (E - 2 if m <= 1.5 else E - 1)
    assert oracle.mx_block_scale_byte(0.0) == 0
    assert oracle.mx_block_scale_byte(np.float32(1e-45)) == 0          # clamped at the bottom of the byte's range
    assert oracle.mx_block_scale_byte(np.float32(3.4e38)) == 126 + 127  # 6 * 2^126 >= FLT_MAX


def test_quantized_values_never_saturate_and_amax_lands_in_the_top_binade():
    x = synth.normal_with_outliers_bf16((64, 256), 0.01, 50.0, 11, 12)
    q = oracle.quantize_mx(synth.bits(x), return_y=True)
    xf = x.float().numpy()
    dec = oracle.dequantize_mx(q)
    for r in range(0, 64, 7):
        for kb in range(8):
            blk = xf[r, kb * 32:(kb + 1) * 32]
            s = oracle.ue8m0_decode(int(q.scales[r, kb]))
            v = np.abs(blk) / s
            assert v.max() <= 6.0 and (v.max() > 3.0 or blk.max() == 0.0)
            # round-to-nearest error bound per element: half the local grid step times the scale
            step = np.where(v < 2, 0.25, np.where(v < 4, 0.5, 1.0))
            assert np.all(np.abs(dec[r, kb * 32:(kb + 1) * 32] - blk) <= step * s + 1e-30)


def test_dequantize_identity_on_grid_and_idempotence():
    rng = np.random.default_rng(3)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    R, C = 8, 128
    vals = rng.choice(grid, size=(R, C)) * rng.choice([-1.0, 1.0], size=(R, C))
    vals[:, ::32] = 6.0  # every block holds its maximum, so the scale is the constructed one
    exps = rng.integers(-6, 6, size=(R, C // 32))
    x = vals * np.repeat(2.0 ** exps, 32, axis=1)
    xb = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)
    assert np.array_equal(xb.float().numpy().astype(np.float64), x), "construction must be exact in bf16"
    q = oracle.quantize_mx(synth.bits(xb))
    assert np.array_equal(q.scales, (exps + 127).astype(np.uint8))
    assert np.array_equal(oracle.dequantize_mx(q), x)
    q2 = oracle.quantize_mx(synth.bits(torch.tensor(oracle.dequantize_mx(q), dtype=torch.float32).to(torch.bfloat16)))
    assert np.array_equal(q2.codes, q.codes) and np.array_equal(q2.scales, q.scales)


def test_colwise_copy_and_2d_blocks():
    x = synth.normal_bf16((64, 96), 1.0, 5)
    xt = x.t().contiguous()
    a = oracle.quantize_mx(synth.bits(x), colwise=True)
    b = oracle.quantize_mx(synth.bits(xt))
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
    # 32 x 32 blocks: one representation for both passes (Section 4.3 at this format's block size)
    w = synth.normal_bf16((64, 96), 0.02, 6)
    row = oracle.quantize_mx(synth.bits(w), block_rows=32)
    col = oracle.quantize_mx(synth.bits(w), block_rows=32, colwise=True)
    assert np.array_equal(oracle.dequantize_mx(row), oracle.dequantize_mx(col).T)
    assert np.array_equal(row.scales[:32, 0], np.full(32, row.scales[0, 0]))
    # with 1 x 32 blocks on both copies the two representations differ on random data
    row1 = oracle.quantize_mx(synth.bits(w))
    col1 = oracle.quantize_mx(synth.bits(w), colwise=True)
    assert not np.array_equal(oracle.dequantize_mx(row1), oracle.dequantize_mx(col1).T)
    with pytest.raises(ValueError):
        oracle.quantize_mx(synth.bits(synth.normal_bf16((16, 48), 1.0, 1)))


def test_hadamard32_structure_and_special_inputs():
    H = np.array([[oracle.hadamard32_entry(j, k) for k in range(32)] for j in range(32)], dtype=np.float64)
    assert np.array_equal(H @ H.T, 32 * np.eye(32)) and np.array_equal(H, H.T)
    H2 = np.array([[1, 1], [1, -1]], dtype=np.float64)
    H16 = np.array([[oracle.hadamard16_entry(j, k) for k in range(16)] for j in range(16)], dtype=np.float64)
    assert np.array_equal(H, np.kron(H2, H16))
    mask = 0xA5C3_73E5
    s = np.array([-1.0 if (mask >> j) & 1 else 1.0 for j in range(32)])
    rng = np.random.default_rng(1)
    x = rng.standard_normal(32).astype(np.float32)
    y = oracle.rht32(x, mask)
    ref = (s * x.astype(np.float64)) @ H / math.sqrt(32.0)
    assert np.allclose(y, ref, rtol=0, atol=1e-6 * np.abs(x).sum())
    assert abs(np.linalg.norm(y.astype(np.float64)) - np.linalg.norm(x.astype(np.float64))) < 1e-5  # Parseval
    back = (y.astype(np.float64) @ H.T / math.sqrt(32.0)) * s  # involution (H symmetric, S its own inverse)
    assert np.allclose(back, x, atol=1e-5)
    one = np.zeros(32, dtype=np.float32)
    one[5] = 2.0
    y = oracle.rht32(one, mask)
    assert np.allclose(y, [2.0 / math.sqrt(32.0) * s[5] * H[5, k] for k in range(32)], rtol=1e-7)
    const = oracle.rht32(np.full(32, 3.0, dtype=np.float32), 0)
    assert np.isclose(const[0], 3.0 * math.sqrt(32.0), rtol=1e-7) and np.all(const[1:] == 0.0)


def test_rht32_cancels_in_the_dot_product_and_scales_live_in_rotated_space():
    rng = np.random.default_rng(2)
    mask = 0x1234_ABCD
    A = rng.standard_normal((4, 64)).astype(np.float32)
    Bm = rng.standard_normal((3, 64)).astype(np.float32)
    rot = lambda M: np.stack([np.concatenate([oracle.rht32(r[c:c + 32], mask) for c in (0, 32)]) for r in M])
    assert np.allclose(rot(A).astype(np.float64) @ rot(Bm).astype(np.float64).T,
                       A.astype(np.float64) @ Bm.astype(np.float64).T, atol=1e-4)
    # a constant chunk grows by sqrt(32) under the transform: its scale must come from the rotated values
    x = torch.full((1, 32), 1.0, dtype=torch.bfloat16)
    q = oracle.quantize_mx(synth.bits(x), rht=True, sign_mask=0, return_y=True)
    assert np.isclose(q.y[0, 0], math.sqrt(32.0), rtol=1e-6)
    assert q.scales[0, 0] == oracle.mx_block_scale_byte(np.float32(q.y[0, 0]))


def test_sr_uses_the_same_draws_and_is_unbiased():
    x = synth.normal_bf16((32, 64), 1.0, 9)
    xf = x.float().numpy().astype(np.float64)
    # element (0, 0): v known, draw known -> decision by the printed rule
    q = oracle.quantize_mx(synth.bits(x), rounding=oracle.SR, seed=0, sr_offset=0, return_y=True)
    s = float(oracle.mx_block_encode_scale(int(q.scales[0, 0])))
    v = np.float32(q.y[0, 0]) * np.float32(s)
    assert (q.codes[0, 0] & 15) == oracle.e2m1_encode_sr(v, oracle.sr_draw(0, 0, 0))
    acc = np.zeros_like(xf)
    S = 512
    for seed in range(S):
        acc += oracle.dequantize_mx(oracle.quantize_mx(synth.bits(x), rounding=oracle.SR, seed=seed))
    scale = np.repeat(np.vectorize(oracle.ue8m0_decode)(q.scales.astype(int)), 32, axis=1)
    step = 2.0 * scale  # widest grid step times the block scale
    assert np.all(np.abs(acc / S - xf) <= step * (1 / 512 + 2 / math.sqrt(S)))


def test_nvfp4_is_the_more_accurate_format_on_the_papers_kind_of_data():
    """Section 2: smaller blocks and a fractional block scale give NVFP4 a lower quantization error than MXFP4.
    Relative L2 error of the decoded tensor on Gaussian data with a few large outliers."""
    x = synth.normal_with_outliers_bf16((128, 1024), 0.001, 100.0, 71, 72)
    xf = x.float().numpy().astype(np.float64)
    nv = oracle.dequantize(oracle.quantize(synth.bits(x)))
    mx = oracle.dequantize_mx(oracle.quantize_mx(synth.bits(x)))
    e_nv = np.linalg.norm(nv - xf) / np.linalg.norm(xf)
    e_mx = np.linalg.norm(mx - xf) / np.linalg.norm(xf)
    assert e_nv < e_mx and e_nv < 0.12 and e_mx < 0.2, (e_nv, e_mx)
    # and MXFP4 wastes part of the grid: the share of elements that land on +-4 or +-6 is lower
    top = lambda codes: np.isin(np.concatenate([codes & 7, (codes >> 4) & 7]), [6, 7]).mean()
    assert top(oracle.quantize_mx(synth.bits(x)).codes) < top(oracle.quantize(synth.bits(x)).codes)
