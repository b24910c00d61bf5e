"""MXFP4 (the paper's comparison format, Section 5 / Appendix B.4) through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def upload_mx(q: oracle.QuantizedMX) -> B.NVFP4Tensor:
    glob = torch.tensor([0.0, 1.0], dtype=torch.float32, device="cuda")
    return B.NVFP4Tensor(torch.from_numpy(np.ascontiguousarray(q.codes)).cuda(),
                         torch.from_numpy(oracle.sf_swizzle(q.scales)).cuda(), glob, q.rows, q.cols, B.SF_SWIZZLED,
                         B.FORMAT_MXFP4)


def run_gemm(a, b, fp32):
    A, Bt = upload_mx(a), upload_mx(b)
    D = torch.full((a.rows, b.rows), float("nan"), dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
    B.nvfp4_gemm(A, Bt, D)
    B.nvfp4_device_status()
    return D.float().cpu().numpy()


def reference(a, b):
    return oracle.gemm_tn(oracle.dequantize_mx(a), oracle.dequantize_mx(b))


def test_gemm_exact_ones_and_block_pairing():
    M, N, K = 256, 256, 512
    ones = lambda R: oracle.QuantizedMX(np.full((R, K // 2), 0x22, np.uint8), np.full((R, K // 32), 127, np.uint8), R, K)
    assert np.array_equal(run_gemm(ones(M), ones(N), True), np.full((M, N), float(K), np.float32))
    # block scales that differ per block and per row: a wrong pairing of scale bytes with 32-element blocks, rows or
    # K-steps changes the exact result (all partial sums are small integers times powers of two)
    rng = np.random.default_rng(5)

    def make(R):
        sc = (127 + rng.integers(-3, 4, size=(R, K // 32))).astype(np.uint8)
        return oracle.QuantizedMX(np.full((R, K // 2), 0x22, np.uint8), sc, R, K)

    a, b = make(M), make(N)
    Dref, _ = reference(a, b)
    assert np.array_equal(run_gemm(a, b, True).astype(np.float64), Dref)


@pytest.mark.parametrize("shape", [(256, 256, 256), (256, 512, 1024), (512, 256, 2048), (768, 512, 768)])
@pytest.mark.parametrize("fp32", [False, True])
def test_gemm_against_fp64_product_of_decoded_operands(shape, fp32):
    M, N, K = shape
    a = oracle.quantize_mx(synth.bits(synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, 31, 32)))
    b = oracle.quantize_mx(synth.bits(synth.normal_bf16((N, K), 0.02, 33)), block_rows=32)
    Dref, T = reference(a, b)
    P.assert_gemm_close(run_gemm(a, b, fp32), Dref, T, not fp32, f"mx gemm {shape}")


def test_gemm_rejects_mixed_formats_and_ragged_mx_shapes():
    a = oracle.quantize_mx(synth.bits(synth.normal_bf16((128, 256), 1.0, 1)))
    A = upload_mx(a)
    D = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(B.NVFP4Error) as e:
        B.nvfp4_gemm(A, A, D)  # M, N = 128: only the CTA-pair kernel handles this format
    assert e.value.status == 8
    n = P.upload(oracle.quantize(synth.bits(synth.normal_bf16((256, 256), 1.0, 2))))
    m = upload_mx(oracle.quantize_mx(synth.bits(synth.normal_bf16((256, 256), 1.0, 3))))
    with pytest.raises(B.NVFP4Error) as e:
        B.nvfp4_gemm(n, m, torch.empty((256, 256), dtype=torch.float32, device="cuda"))
    assert e.value.status == 4
