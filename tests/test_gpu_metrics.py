"""Parity of the quantization-error reductions (Appendix E.2) with the oracle's binary64 sums, through the C ABI.

Tolerance: the kernel decodes in FP32 (two roundings, 2^-23 relative on x^), squares in FP32 per 16 elements and
sums in FP64; the sums agree with binary64 to a few 1e-6 relative.  1e-5 is asserted."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def close(got, want, rel=1e-5):
    return abs(got - want) <= rel * abs(want) + 1e-300


@pytest.mark.parametrize("shape", [(128, 64), (384, 1088), (2048, 5120)])
@pytest.mark.parametrize("block_rows,rounding", [(1, oracle.RNE), (16, oracle.RNE), (1, oracle.SR)])
@pytest.mark.parametrize("sf_layout", [B.SF_LINEAR, B.SF_SWIZZLED])
def test_quant_error_of_an_oracle_made_copy(shape, block_rows, rounding, sf_layout):
    x = synth.normal_with_outliers_bf16(shape, 0.01, 30.0, 3, 4)
    q = oracle.quantize(synth.bits(x), block_rows=block_rows, rounding=rounding, seed=5)
    err_ref, n_ref = oracle.quant_error(x.float().numpy(), oracle.dequantize(q))
    t = P.upload(q) if sf_layout == B.SF_SWIZZLED else P.upload_linear(q)
    out = B.nvfp4_quant_error(x.cuda(), t).cpu().numpy()
    assert close(out[0], err_ref) and close(out[1], n_ref), (out, err_ref, n_ref)


def test_quant_error_mxfp4_and_leading_dimension():
    big = synth.normal_bf16((256, 640), 1.0, 7)
    x = big[:, 128:640]  # ld 640, 32-byte aligned start
    q = oracle.quantize_mx(synth.bits(x.contiguous()))
    err_ref, n_ref = oracle.quant_error(x.float().numpy(), oracle.dequantize_mx(q))
    g = P.gpu_quantize_mx(x.contiguous().cuda(), rowwise=True)[0]
    out = B.nvfp4_quant_error(big.cuda()[:, 128:640], g).cpu().numpy()
    assert close(out[0], err_ref) and close(out[1], n_ref)
    assert err_ref / n_ref > 5e-3  # the power-of-two scale costs accuracy (Appendix B.4)


def test_quant_error_is_zero_on_the_grid_and_ranks_formats():
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    rng = np.random.default_rng(2)
    v = rng.choice(grid, size=(128, 256)) * rng.choice([-1.0, 1.0], size=(128, 256))
    v[:, ::16] = 6.0
    xb = torch.tensor(v, dtype=torch.float32).to(torch.bfloat16).cuda()
    g = P.gpu_quantize(xb, rowwise=True)[0]
    out = B.nvfp4_quant_error(xb, g).cpu().numpy()
    assert out[0] <= 1e-12 * out[1] and close(out[1], float(np.sum(v * v)), 1e-12)
    # Section 2: NVFP4 is the more accurate format on data with outliers
    x = synth.normal_with_outliers_bf16((256, 1024), 0.001, 100.0, 71, 72).cuda()
    e_nv = B.nvfp4_quant_error(x, P.gpu_quantize(x, rowwise=True)[0]).cpu().numpy()
    e_mx = B.nvfp4_quant_error(x, P.gpu_quantize_mx(x, rowwise=True)[0]).cpu().numpy()
    assert e_nv[0] < e_mx[0] and e_nv[1] == e_mx[1]


@pytest.mark.parametrize("ref_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("test_dtype", [torch.bfloat16, torch.float32])
def test_sq_error_between_dense_tensors(ref_dtype, test_dtype):
    g = torch.Generator().manual_seed(11)
    a = torch.randn((300, 1000 + 8), generator=g).to(ref_dtype)[:, :1000]
    b = (a.float() + 0.01 * torch.randn((300, 1000), generator=g)).to(test_dtype)
    err_ref, n_ref = oracle.quant_error(a.float().numpy(), b.float().numpy())
    out = B.nvfp4_sq_error(a.cuda(), b.cuda()).cpu().numpy()
    assert close(out[0], err_ref) and close(out[1], n_ref)
    assert np.array_equal(B.nvfp4_sq_error(a.cuda(), a.cuda())[:1].cpu().numpy(), [0.0])


def test_wgrad_error_of_the_fp4_layer_against_the_bf16_layer():
    """The use Appendix E.2 has in mind: relative error of the FP4 weight gradient, measured against the BF16 one,
    with every product on the GPU.  The value must match the oracle's for the same operands."""
    M, N, K = 512, 256, 256
    x = synth.normal_with_outliers_bf16((M, K), 0.01, 20.0, 31, 32)
    dy = synth.normal_bf16((M, N), 0.02, 33)
    mask = 0x73E5
    xq = oracle.quantize(synth.bits(x), colwise=True, rht=True, sign_mask=mask)
    gq = oracle.quantize(synth.bits(dy), colwise=True, rht=True, sign_mask=mask)  # RNE: deterministic reference
    dW4 = torch.empty((N, K), dtype=torch.float32, device="cuda")
    B.nvfp4_gemm(P.upload(gq), P.upload(xq), dW4)
    dW16 = torch.empty((N, K), dtype=torch.float32, device="cuda")
    B.nvfp4_linear_bf16_bwd(dy.cuda(), x.cuda(), None, K, None, dW16)
    out = B.nvfp4_sq_error(dW16, dW4).cpu().numpy()
    ref4 = oracle.gemm_tn(oracle.dequantize(gq), oracle.dequantize(xq), want_T=False)
    (_, _), (ref16, _) = oracle.linear_bf16_bwd(synth.bits(dy), synth.bits(x), synth.bits(torch.zeros((N, K), dtype=torch.bfloat16)))
    err_ref, n_ref = oracle.quant_error(ref16, ref4)
    assert close(out[0], err_ref, 1e-3) and close(out[1], n_ref, 1e-4), (out, err_ref, n_ref)
    assert 1e-3 < out[0] / out[1] < 0.2
