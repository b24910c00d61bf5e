"""Parity of the single-pass quantizer with a global scale per row (Appendix B.1, closing remark) and of the GEMM
that applies the scale vectors in its epilogue, against the oracle (each row quantized as a tensor of its own),
through the C ABI.  No transform is involved: codes, scale bytes and the per-row words are compared bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def gpu_rowscale(x, sf_layout=B.SF_SWIZZLED, **opt):
    R, C = x.shape
    t = B.alloc_tensor(R, C, sf_layout, format=B.FORMAT_NVFP4_ROWSCALE)
    B.nvfp4_quantize(x.cuda(), B.quant_opts(**opt), t, None)
    torch.cuda.synchronize()
    return t


def download_rows(t):
    codes = t.codes.cpu().numpy()
    sc = t.scales.cpu().numpy()
    scales = oracle.sf_unswizzle(sc, t.rows, t.cols // 16) if t.sf_layout == B.SF_SWIZZLED else sc.reshape(t.rows, -1)
    return codes, scales, t.glob.cpu().numpy().reshape(t.rows, 2)


def assert_rows_exact(t, ref, what=""):
    codes, scales, glob = download_rows(t)
    assert glob.view(np.uint32).tolist() == ref.glob.view(np.uint32).tolist(), f"{what}: per-row words"
    assert np.array_equal(scales, ref.scales), f"{what}: scale bytes"
    assert np.array_equal(codes, ref.codes), f"{what}: codes"


@pytest.mark.parametrize("shape", [(128, 64), (256, 5120), (128, 5184), (128, 10240), (256, 20480), (128, 20544)])
@pytest.mark.parametrize("rounding", [oracle.RNE, oracle.SR])
def test_quantizer_bit_exact(shape, rounding):
    # rows of up to 5120 / 10240 / 20480 elements live in the registers of 1 / 2 / 4 warps; 20544 takes the two-sweep kernel
    x = synth.normal_with_outliers_bf16(shape, 0.01, 40.0, 11, 12)
    x[5] = 0  # an all-zero row: s_enc = 1, scales 0
    x[7] *= 1e-3
    t = gpu_rowscale(x, rounding=rounding, seed=3, sr_offset=9)
    assert_rows_exact(t, oracle.quantize_rowscale(synth.bits(x), rounding=rounding, seed=3, sr_offset=9), f"{shape}")


def test_linear_scale_layout_ragged_rows_and_argument_checks():
    x = synth.normal_bf16((48, 208), 1.0, 21)  # rows not a multiple of 8 warps x n, cols not of 512
    t = gpu_rowscale(x, sf_layout=B.SF_LINEAR)
    assert_rows_exact(t, oracle.quantize_rowscale(synth.bits(x)), "linear layout")
    xd = x.cuda()
    t2 = B.alloc_tensor(48, 208, B.SF_LINEAR, format=B.FORMAT_NVFP4_ROWSCALE)
    col = B.alloc_tensor(208, 48, B.SF_LINEAR, format=B.FORMAT_NVFP4_ROWSCALE)
    with pytest.raises(B.NVFP4Error):  # no transposed copy in this format
        B.nvfp4_quantize(xd, B.quant_opts(), t2, col)
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_quantize(xd, B.quant_opts(block_rows=16), t2, None)
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_quantize(xd, B.quant_opts(rht_rowwise=True), t2, None)


def upload_rows(q):
    return B.NVFP4Tensor(torch.from_numpy(np.ascontiguousarray(q.codes)).cuda(),
                         torch.from_numpy(oracle.sf_swizzle(q.scales)).cuda(),
                         torch.from_numpy(np.ascontiguousarray(q.glob).reshape(-1)).cuda(), q.rows, q.cols,
                         B.SF_SWIZZLED, B.FORMAT_NVFP4_ROWSCALE)


@pytest.mark.parametrize("fp32", [False, True])
@pytest.mark.parametrize("a_rows,b_rows", [(True, False), (False, True), (True, True)])
def test_gemm_applies_the_scale_vectors(a_rows, b_rows, fp32):
    M, N, K = 512, 768, 1024
    xa = synth.normal_with_outliers_bf16((M, K), 0.01, 40.0, 31, 32)
    xa[::3] *= 64.0   # rows of very different magnitude: a wrong or missing row factor is far outside the bound
    xb = synth.normal_bf16((N, K), 0.02, 33)
    xb[1::2] *= 0.01
    if a_rows:
        qa = oracle.quantize_rowscale(synth.bits(xa)); A = upload_rows(qa); da = oracle.dequantize_rowscale(qa)
    else:
        qa = oracle.quantize(synth.bits(xa)); A = P.upload(qa); da = oracle.dequantize(qa)
    if b_rows:
        qb = oracle.quantize_rowscale(synth.bits(xb)); Bt = upload_rows(qb); db = oracle.dequantize_rowscale(qb)
    else:
        qb = oracle.quantize(synth.bits(xb), block_rows=16); Bt = P.upload(qb); db = oracle.dequantize(qb)
    Dref, T = oracle.gemm_tn(da, db)
    D = torch.full((M, N), float("nan"), dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
    B.nvfp4_gemm(A, Bt, D)
    B.nvfp4_device_status()
    P.assert_gemm_close(D.float().cpu().numpy(), Dref, T, not fp32, f"rows A={a_rows} B={b_rows}")
    if fp32:  # accumulation into an fp32 output goes through the same epilogue
        D0 = torch.randn((M, N), generator=torch.Generator().manual_seed(1))
        D2 = D0.cuda()
        B.nvfp4_gemm(A, Bt, D2, True)
        P.assert_gemm_close(D2.cpu().numpy(), Dref + D0.numpy().astype(np.float64), T + np.abs(D0.numpy()), False, "accumulate")


def test_row_scales_keep_small_rows_alive_next_to_an_outlier_row_and_metric_agrees():
    """What the finer granularity buys besides the saved pass: one huge token no longer flushes the others."""
    x = synth.normal_bf16((256, 512), 1e-3, 41)
    x[17] *= 3e7
    xd = x.cuda()
    t_rows = gpu_rowscale(x)
    t_tensor = P.gpu_quantize(x, rowwise=True)[0]
    e_rows = B.nvfp4_quant_error(xd, t_rows).cpu().numpy()
    e_tensor = B.nvfp4_quant_error(xd, t_tensor).cpu().numpy()
    xf = x.float().numpy().astype(np.float64)
    ref = oracle.quant_error(xf, oracle.dequantize_rowscale(oracle.quantize_rowscale(synth.bits(x))))
    assert abs(e_rows[0] - ref[0]) <= 1e-5 * ref[0] and abs(e_rows[1] - ref[1]) <= 1e-5 * ref[1]
    # decode (test aid) agrees with the oracle's decode
    dec = B.nvfp4_dequantize(t_rows).cpu().numpy()
    assert np.allclose(dec, oracle.dequantize_rowscale(oracle.quantize_rowscale(synth.bits(x))), rtol=1e-6, atol=0)
    small = np.arange(256) != 17
    err_rows = np.abs(dec - xf)[small].max()
    err_tensor = np.abs(B.nvfp4_dequantize(t_tensor).cpu().numpy() - xf)[small].max()
    assert err_rows < 0.2 * np.abs(xf[small]).max() and err_tensor == np.abs(xf[small]).max()


def test_forward_only_layer_with_row_scaled_activations():
    """nvfp4_linear_fwd with NVFP4_LINEAR_ROW_SCALES: X quantized in one pass with a scale per token, W with 16x16
    blocks and its tensor scale, Fprop applying the token vector in its epilogue."""
    M, N, K = 512, 768, 1024
    x = synth.normal_with_outliers_bf16((M, K), 0.01, 40.0, 51, 52)
    x[::5] *= 100.0
    w = synth.normal_bf16((N, K), 0.02, 53)
    W_row = B.alloc_tensor(N, K)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    o = B.quant_opts(flags=B.LINEAR_ROW_SCALES)
    B.nvfp4_linear_fwd(x.cuda(), w.cuda(), o, Y, None, W_row, None, False, ws)
    B.nvfp4_device_status()
    qa = oracle.quantize_rowscale(synth.bits(x))
    qb = oracle.quantize(synth.bits(w), block_rows=16)
    Dref, T = oracle.gemm_tn(oracle.dequantize_rowscale(qa), oracle.dequantize(qb))
    P.assert_gemm_close(Y.float().cpu().numpy(), Dref, T, True, "forward-only layer")
    with pytest.raises(B.NVFP4Error):  # a saved transposed copy cannot be made with row scales
        B.nvfp4_linear_fwd(x.cuda(), w.cuda(), o, Y, B.alloc_tensor(K, M), W_row, None, False, ws)
