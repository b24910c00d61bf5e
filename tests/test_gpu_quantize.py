"""Parity of the CUDA quantizer (through the C ABI) with the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu
MASK = synth.DEFAULT_RHT_SIGN_MASK


def rand_bf16(shape, seed, std=1.0, outliers=0.0):
    if outliers:
        return synth.normal_with_outliers_bf16(shape, outliers, 50.0, seed, seed + 1)
    return synth.normal_bf16(shape, std, seed)


SHAPES = [(128, 128), (256, 384), (512, 1024)]          # full tiles (swizzled scale layout)
RAGGED = [(16, 16), (144, 208), (48, 400), (272, 16)]   # partial tiles (linear scale layout)


@pytest.mark.parametrize("shape", SHAPES + RAGGED)
@pytest.mark.parametrize("which", ["row", "col", "both"])
def test_rne_1x16_is_bit_exact(shape, which):
    x = rand_bf16(shape, 100 + shape[0], outliers=0.01)
    layout = B.SF_SWIZZLED if shape in SHAPES else B.SF_LINEAR
    row, col = P.gpu_quantize(x, rowwise=which != "col", colwise=which != "row", sf_layout=layout)
    if row is not None:
        P.assert_exact(row, oracle.quantize(synth.bits(x)), f"row {shape}")
    if col is not None:
        P.assert_exact(col, oracle.quantize(synth.bits(x), colwise=True), f"col {shape}")


@pytest.mark.parametrize("shape", [(128, 128), (1024, 1024), (48, 80), (144, 208)])
@pytest.mark.parametrize("which", ["row", "col", "both"])
def test_rne_16x16_weights_are_bit_exact_and_consistent(shape, which):
    w = rand_bf16(shape, 7, std=0.02)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    row, col = P.gpu_quantize(w, rowwise=which != "col", colwise=which != "row", sf_layout=layout, block_rows=16)
    if row is not None:
        P.assert_exact(row, oracle.quantize(synth.bits(w), block_rows=16), "W row")
    if col is not None:
        P.assert_exact(col, oracle.quantize(synth.bits(w), block_rows=16, colwise=True), "W col")
    if row is not None and col is not None:
        # Section 4.3: one quantized representation for both passes
        assert torch.equal(B.nvfp4_dequantize(row), B.nvfp4_dequantize(col).T.contiguous())


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (144, 208)])
@pytest.mark.parametrize("which", ["row", "col", "both"])
@pytest.mark.parametrize("independent", [False, True])
def test_stochastic_rounding_is_bit_exact_given_the_stream(shape, which, independent):
    x = rand_bf16(shape, 31, std=1e-3)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    seed, off = 0x1234_5678_9ABC_DEF0, (3 << 32) | 17
    row, col = P.gpu_quantize(x, rowwise=which != "col", colwise=which != "row", sf_layout=layout,
                              rounding=B.ROUND_STOCHASTIC, seed=seed, sr_offset=off,
                              flags=B.SR_INDEPENDENT_COPIES if independent else 0)
    if row is not None:
        P.assert_exact(row, oracle.quantize(synth.bits(x), rounding=oracle.SR, seed=seed, sr_offset=off), "SR row")
    if col is not None:
        off_c = off | (1 << 63) if independent else off
        P.assert_exact(col, oracle.quantize(synth.bits(x), colwise=True, rounding=oracle.SR, seed=seed,
                                            sr_offset=off_c), "SR col")


def test_sr_16x16_and_seed_zero():
    w = rand_bf16((128, 256), 5, std=0.02)
    row, col = P.gpu_quantize(w, colwise=True, block_rows=16, rounding=B.ROUND_STOCHASTIC)
    P.assert_exact(row, oracle.quantize(synth.bits(w), block_rows=16, rounding=oracle.SR), "2D SR row")
    P.assert_exact(col, oracle.quantize(synth.bits(w), block_rows=16, rounding=oracle.SR, colwise=True), "2D SR col")


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (144, 208)])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_rht_copies_follow_the_tolerance_protocol(shape, rounding):
    x = rand_bf16(shape, 55, outliers=0.01)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    row, col = P.gpu_quantize(x, colwise=True, sf_layout=layout, rht_rowwise=True, rht_colwise=True,
                              rht_sign_mask=MASK, rounding=rounding, seed=9, sr_offset=1)
    xd = x.cuda()
    y_row = B.nvfp4_rht16(xd, False, MASK).cpu().numpy()
    y_col = B.nvfp4_rht16(xd, True, MASK).cpu().numpy()
    s1 = P.assert_rht_close(synth.bits(x), row, y_row, colwise=False, sign_mask=MASK, rounding=rounding, seed=9,
                            sr_offset=1, what="RHT row")
    s2 = P.assert_rht_close(synth.bits(x), col, y_col, colwise=True, sign_mask=MASK, rounding=rounding, seed=9,
                            sr_offset=1, what="RHT col")
    assert s1["excused_codes"] + s2["excused_codes"] <= 1e-3 * 2 * x.numel()


def test_recipe_combination_row_plain_col_rht():
    # the activation recipe: row-wise copy untouched (bit-exact), column-wise copy rotated (tolerance)
    x = rand_bf16((256, 256), 77, outliers=0.01)
    row, col = P.gpu_quantize(x, colwise=True, rht_colwise=True, rht_sign_mask=MASK)
    P.assert_exact(row, oracle.quantize(synth.bits(x)), "row of mixed call")
    y_col = B.nvfp4_rht16(x.cuda(), True, MASK).cpu().numpy()
    P.assert_rht_close(synth.bits(x), col, y_col, colwise=True, sign_mask=MASK, rounding=oracle.RNE, what="col of mixed")


def test_degenerate_inputs():
    z = torch.zeros((128, 128), dtype=torch.bfloat16)
    row, col = P.gpu_quantize(z, colwise=True)
    P.assert_exact(row, oracle.quantize(synth.bits(z)), "zeros row")
    P.assert_exact(col, oracle.quantize(synth.bits(z), colwise=True), "zeros col")
    # tiny and huge magnitudes, blocks that underflow the E4M3 range, negative zero
    x = rand_bf16((128, 128), 3)
    x[0, :16] = 3.0e38
    x[5, 32:48] = 1e-30
    x[7, 0] = -0.0
    row, col = P.gpu_quantize(x, colwise=True)
    P.assert_exact(row, oracle.quantize(synth.bits(x)), "extremes row")
    P.assert_exact(col, oracle.quantize(synth.bits(x), colwise=True), "extremes col")
    # leading dimension larger than the row length
    wide = rand_bf16((128, 256), 4).cuda()
    sub = wide[:, :128]
    r = B.alloc_tensor(128, 128)
    B.nvfp4_quantize(sub, B.quant_opts(), r, None)
    P.assert_exact(r, oracle.quantize(synth.bits(wide.cpu())[:, :128]), "strided input")
    # provided amax
    r2 = B.alloc_tensor(128, 128)
    r2.glob[0] = r.glob[0]
    B.nvfp4_quantize(sub, B.quant_opts(flags=B.AMAX_PROVIDED), r2, None)
    P.assert_exact(r2, oracle.quantize(synth.bits(wide.cpu())[:, :128]), "amax provided")


@pytest.mark.parametrize("scale", [1e-30, 1e-36, 3e-39, 1e30])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_extreme_magnitudes_stay_bit_exact(scale, rounding):
    """Whole tensors near the ends of the bf16 range: the global encode scale clamps at FLT_MAX (amax below
    2688 / FLT_MAX), block amaxes are denormal (the exact-division path of amax_b / 6), products land in the
    denormal range (no flush to zero anywhere), and at the top 2688 / amax is itself tiny."""
    x = (synth.normal_bf16((128, 256), 1.0, 21).float() * scale).to(torch.bfloat16)
    x[3, 16:32] = 0.0
    for block_rows in (1, 16):
        row, col = P.gpu_quantize(x, colwise=True, block_rows=block_rows, rounding=rounding, seed=5, sr_offset=9)
        kw = dict(block_rows=block_rows, rounding=rounding, seed=5, sr_offset=9)
        P.assert_exact(row, oracle.quantize(synth.bits(x), **kw), f"row scale {scale} blocks {block_rows}")
        P.assert_exact(col, oracle.quantize(synth.bits(x), colwise=True, **kw), f"col scale {scale} blocks {block_rows}")


def test_gpu_sr_is_unbiased_over_seeds():
    x = rand_bf16((128, 128), 8, std=1e-3)
    xd = x.cuda()
    S = 512
    acc = torch.zeros((128, 128), dtype=torch.float64, device="cuda")
    acc_c = torch.zeros((128, 128), dtype=torch.float64, device="cuda")
    row, col = B.alloc_tensor(128, 128), B.alloc_tensor(128, 128)
    for seed in range(S):
        B.nvfp4_quantize(xd, B.quant_opts(rounding=B.ROUND_STOCHASTIC, seed=seed), row, col)
        acc += B.nvfp4_dequantize(row).double()
        acc_c += B.nvfp4_dequantize(col).double().T
    ref = oracle.quantize(synth.bits(x))
    sb = np.vectorize(oracle.e4m3_decode)(ref.scales).repeat(16, axis=1) * float(ref.s_dec)
    xf = x.double().numpy()
    sat = np.maximum(np.abs(xf) - 6.0 * sb, 0.0)
    assert np.all(np.abs(acc.cpu().numpy() / S - xf) <= sat + 2.0 * sb * (1 / 512 + 2.5 / np.sqrt(S)) + 1e-12)
    refc = oracle.quantize(synth.bits(x), colwise=True)
    sbc = (np.vectorize(oracle.e4m3_decode)(refc.scales).repeat(16, axis=1) * float(refc.s_dec)).T
    satc = np.maximum(np.abs(xf) - 6.0 * sbc, 0.0)
    assert np.all(np.abs(acc_c.cpu().numpy() / S - xf) <= satc + 2.0 * sbc * (1 / 512 + 2.5 / np.sqrt(S)) + 1e-12)


def test_config1_tensors_all_roles():
    p = synth.config1()
    # X: row-wise plain + column-wise rotated, RNE
    row, col = P.gpu_quantize(p.X, colwise=True, rht_colwise=True, rht_sign_mask=p.rht_sign_mask)
    P.assert_exact(row, oracle.quantize(synth.bits(p.X)), "cfg1 X row")
    P.assert_rht_close(synth.bits(p.X), col, B.nvfp4_rht16(p.X.cuda(), True, p.rht_sign_mask).cpu().numpy(),
                       colwise=True, sign_mask=p.rht_sign_mask, rounding=oracle.RNE, what="cfg1 X col")
    # W: 16x16 both copies
    row, col = P.gpu_quantize(p.W, colwise=True, block_rows=16)
    P.assert_exact(row, oracle.quantize(synth.bits(p.W), block_rows=16), "cfg1 W row")
    P.assert_exact(col, oracle.quantize(synth.bits(p.W), block_rows=16, colwise=True), "cfg1 W col")
    # dY: SR, row-wise plain + column-wise rotated
    row, col = P.gpu_quantize(p.dY, colwise=True, rht_colwise=True, rht_sign_mask=p.rht_sign_mask,
                              rounding=B.ROUND_STOCHASTIC, seed=p.sr_seed, sr_offset=p.sr_offset)
    P.assert_exact(row, oracle.quantize(synth.bits(p.dY), rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset),
                   "cfg1 dY row")
    P.assert_rht_close(synth.bits(p.dY), col, B.nvfp4_rht16(p.dY.cuda(), True, p.rht_sign_mask).cpu().numpy(),
                       colwise=True, sign_mask=p.rht_sign_mask, rounding=oracle.SR, seed=p.sr_seed,
                       sr_offset=p.sr_offset, what="cfg1 dY col")


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (144, 208)])
@pytest.mark.parametrize("block_rows", [1, 16])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_binary32_source_is_bit_exact(shape, block_rows, rounding):
    """Appendix B: the source may be FP32 (e.g. master weights).  Values with full 24-bit mantissas."""
    g = torch.Generator().manual_seed(77)
    x = torch.randn(shape, generator=g, dtype=torch.float32) * 0.02
    x[3, 5] = 1.2345678  # the amax, not representable in bf16
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    R, C = shape
    row, col = B.alloc_tensor(R, C, layout), B.alloc_tensor(C, R, layout)
    B.nvfp4_quantize(x.cuda(), B.quant_opts(block_rows=block_rows, rounding=rounding, seed=11, sr_offset=2), row, col)
    kw = dict(block_rows=block_rows, rounding=rounding, seed=11, sr_offset=2)
    P.assert_exact(row, oracle.quantize(x.numpy(), **kw), "f32 row")
    P.assert_exact(col, oracle.quantize(x.numpy(), colwise=True, **kw), "f32 col")
    only = B.alloc_tensor(C, R, layout)
    B.nvfp4_quantize(x.cuda(), B.quant_opts(block_rows=block_rows, rounding=rounding, seed=11, sr_offset=2), None, only)
    P.assert_exact(only, oracle.quantize(x.numpy(), colwise=True, **kw), "f32 col only")
    with pytest.raises(B.NVFP4Error) as e:  # no transform on a binary32 source
        B.nvfp4_quantize(x.cuda(), B.quant_opts(rht_colwise=True, rht_sign_mask=MASK), row, col)
    assert e.value.status == 8
