"""Parity of the quantizer with the other transform sizes of Appendix E.4.2 (d = 2, 4, 8, 128) against the oracle,
through the C ABI: the untransformed copy of a call bit for bit, the transformed one through the tolerance protocol
(the device adds in FP32 in butterfly order, the oracle in binary64)."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu

MASK128 = 0x5A5A_73E5_1234_ABCD_0F0F_3C3C_9999_73E5


def mask_for(d):
    return MASK128 & ((1 << d) - 1)


@pytest.mark.parametrize("d", [2, 4, 8, 128])
@pytest.mark.parametrize("rounding", [oracle.RNE, oracle.SR])
def test_wgrad_operand_recipe_with_another_transform_size(d, rounding):
    """The recipe's use: plain row-wise copy + transformed transposed copy from one call."""
    x = synth.normal_with_outliers_bf16((384, 256), 0.01, 40.0, 50 + d, 51 + d)
    m = mask_for(d)
    row, col = P.gpu_quantize(x, rowwise=True, colwise=True, rht_colwise=True, rht_sign_mask=m, rht_dim=d,
                              rounding=rounding, seed=9, sr_offset=3)
    P.assert_exact(row, oracle.quantize(synth.bits(x), rounding=rounding, seed=9, sr_offset=3), "plain row copy")
    s = P.assert_rht_close(synth.bits(x), col, None, colwise=True, sign_mask=m, rounding=rounding, seed=9, sr_offset=3,
                           what=f"col d={d}", rht_dim=d)
    assert s["excused_codes"] + 16 * s["excused_scales"] <= 1e-3 * s["elements"]


@pytest.mark.parametrize("d", [2, 4, 8, 128])
def test_rowwise_transform_and_both_copies(d):
    x = synth.normal_with_outliers_bf16((256, 384), 0.01, 40.0, 60 + d, 61 + d)
    m = mask_for(d)
    row, col = P.gpu_quantize(x, rowwise=True, colwise=True, rht_rowwise=True, rht_colwise=True, rht_sign_mask=m,
                              rht_dim=d, sf_layout=B.SF_LINEAR)
    P.assert_rht_close(synth.bits(x), row, None, colwise=False, sign_mask=m, rounding=oracle.RNE, what=f"row d={d}",
                       rht_dim=d)
    P.assert_rht_close(synth.bits(x), col, None, colwise=True, sign_mask=m, rounding=oracle.RNE, what=f"col d={d}",
                       rht_dim=d)
    # a single copy on its own
    only_col = P.gpu_quantize(x, rowwise=False, colwise=True, rht_colwise=True, rht_sign_mask=m, rht_dim=d)[1]
    P.assert_rht_close(synth.bits(x), only_col, None, colwise=True, sign_mask=m, rounding=oracle.RNE,
                       what=f"col alone d={d}", rht_dim=d)


@pytest.mark.parametrize("d", [4, 16])
def test_exact_transforms_are_bit_exact(d):
    """Small integers: the rotated values are exact at every stage for d = 4 (and for the recipe's 16), so the
    transformed copy must equal the oracle's (the sign of a zero result aside: a chunk of zeros with flipped signs sums to
    -0 in the butterfly and to +0 in the oracle's running sum)."""
    rng = np.random.default_rng(5)
    x = torch.tensor(rng.integers(-3, 4, size=(128, 256)).astype(np.float32)).to(torch.bfloat16)
    m = 0x73E5 & ((1 << d) - 1)
    row, col = P.gpu_quantize(x, rowwise=True, colwise=True, rht_rowwise=True, rht_colwise=True, rht_sign_mask=m,
                              rht_dim=d)
    P.assert_exact_up_to_zero_sign(row, oracle.quantize(synth.bits(x), rht=True, sign_mask=m, rht_dim=d), "row")
    P.assert_exact_up_to_zero_sign(col, oracle.quantize(synth.bits(x), colwise=True, rht=True, sign_mask=m, rht_dim=d), "col")


def test_ragged_tiles_small_sizes_and_argument_checks():
    x = synth.normal_bf16((144, 208), 1.0, 77)  # neither dimension a multiple of 128
    m = mask_for(8)
    row, col = P.gpu_quantize(x, rowwise=True, colwise=True, rht_colwise=True, rht_sign_mask=m, rht_dim=8,
                              sf_layout=B.SF_LINEAR)
    P.assert_exact(row, oracle.quantize(synth.bits(x)), "plain row copy")
    P.assert_rht_close(synth.bits(x), col, None, colwise=True, sign_mask=m, rounding=oracle.RNE, what="ragged", rht_dim=8)
    xd = x.cuda()
    col = B.alloc_tensor(208, 144, B.SF_LINEAR)
    with pytest.raises(B.NVFP4Error):  # 128-chunks must fit the contraction dimension
        B.nvfp4_quantize(xd, B.quant_opts(rht_colwise=True, rht_dim=128), None, col)
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_quantize(xd, B.quant_opts(rht_colwise=True, rht_dim=3), None, col)
    with pytest.raises(B.NVFP4Error):  # no transform on 16x16 blocks, whatever its size
        B.nvfp4_quantize(xd, B.quant_opts(block_rows=16, rht_colwise=True, rht_dim=4), None, col)


def test_larger_transform_lowers_the_rotated_amax_and_the_gemm_still_cancels():
    """Appendix E.4.2's intuition (a larger matrix spreads an outlier further) and Section 4.2's identity (the two
    rotations cancel in the Wgrad product), end to end on the GPU for d = 128."""
    M, N, K = 256, 256, 128  # Wgrad: dW[N x K] = dY^T X, contraction over M
    x = synth.normal_with_outliers_bf16((M, K), 0.002, 60.0, 81, 82)
    dy = synth.normal_bf16((M, N), 0.05, 83)
    amax = {}
    for d in (4, 128):
        m = mask_for(d)
        xc = P.gpu_quantize(x, rowwise=False, colwise=True, rht_colwise=True, rht_sign_mask=m, rht_dim=d)[1]
        gc = P.gpu_quantize(dy, rowwise=False, colwise=True, rht_colwise=True, rht_sign_mask=m, rht_dim=d)[1]
        amax[d] = float(xc.glob.cpu()[0])
        dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
        B.nvfp4_gemm(gc, xc, dW)
        B.nvfp4_device_status()
        (_, _), (ref, T) = oracle.linear_bf16_bwd(synth.bits(dy), synth.bits(x), synth.bits(torch.zeros((N, K), dtype=torch.bfloat16)))
        rel = np.linalg.norm(dW.cpu().numpy() - ref) / np.linalg.norm(ref)
        assert rel < 0.25, (d, rel)  # FP4 noise only: a transform that did not cancel would give rel ~ 1
    assert amax[128] < amax[4]


@pytest.mark.parametrize("d", [4, 128])
def test_linear_layer_with_another_transform_size(d):
    """nvfp4_linear_fwd / _bwd pass rht_dim through to both Wgrad operands: dW must match the product of the
    oracle's operands made with the same size (and would be far off if only one side used it)."""
    M, N, K = 256, 256, 256
    x = synth.normal_with_outliers_bf16((M, K), 0.01, 20.0, 71, 72)
    w = synth.normal_bf16((N, K), 0.02, 73)
    dy = synth.normal_bf16((M, N), 0.01, 74)
    m = mask_for(d)
    o = B.quant_opts(rht_sign_mask=m, rht_dim=d, seed=5, sr_offset=1)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    B.nvfp4_linear_fwd(x.cuda(), w.cuda(), o, Y, X_col, W_row, W_col, False, ws_f)
    B.nvfp4_linear_bwd(dy.cuda(), X_col, W_col, K, o, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    P.assert_rht_close(synth.bits(x), X_col, None, colwise=True, sign_mask=m, rounding=oracle.RNE, what="X col", rht_dim=d)
    gx = oracle.quantize(synth.bits(x), colwise=True, rht=True, sign_mask=m, rht_dim=d, amax_override=float(X_col.glob.cpu()[0]))
    # the layer's dY copy lives in its workspace: remake it with the same options to learn its amax (protocol)
    g_col = B.alloc_tensor(N, M)
    B.nvfp4_quantize(dy.cuda(), B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=m, rht_dim=d,
                                             seed=5, sr_offset=1), None, g_col)
    gg = oracle.quantize(synth.bits(dy), colwise=True, rht=True, sign_mask=m, rht_dim=d, rounding=oracle.SR, seed=5,
                         sr_offset=1, amax_override=float(g_col.glob.cpu()[0]))
    Dref, T = oracle.gemm_tn(oracle.dequantize(gg), oracle.dequantize(gx))
    err = np.abs(dW.cpu().numpy() - Dref)
    assert np.count_nonzero(err > 1e-3 * T + 1e-30) <= 1e-3 * err.size and np.all(err <= 2e-2 * T + 1e-30)
