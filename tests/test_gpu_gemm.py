"""Parity of the tcgen05 block-scaled GEMM (through the C ABI) with the FP64 product of the decoded operands."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def operands(M, N, K, seed):
    a = oracle.quantize(synth.bits(synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, seed, seed + 1)))
    b = oracle.quantize(synth.bits(synth.normal_bf16((N, K), 0.02, seed + 2)), block_rows=16)
    return a, b


def run_gemm(a, b, fp32, tile_n, accumulate=False, D0=None):
    B.nvfp4_set_gemm_tile_n(tile_n)
    try:
        A, Bt = P.upload(a), P.upload(b)
        D = torch.full((a.rows, b.rows), float("nan"), dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
        if D0 is not None:
            D.copy_(D0)
        B.nvfp4_gemm(A, Bt, D, accumulate)
        B.nvfp4_device_status()
        return D.float().cpu().numpy()
    finally:
        B.nvfp4_set_gemm_tile_n(0)


@pytest.mark.parametrize("tile_n", [128, 256, 512, 768])
def test_exact_all_ones(tile_n):
    # every code 1.0 (nibble 2), every block scale 1.0 (0x38), tensor scales 1: each output = K exactly
    M, N, K = 256, 256, 512
    q = lambda R: oracle.Quantized(np.full((R, K // 2), 0x22, np.uint8), np.full((R, K // 16), 0x38, np.uint8),
                                   np.array([1.0, 1.0], np.float32), R, K)
    D = run_gemm(q(M), q(N), True, tile_n)
    assert np.array_equal(D, np.full((M, N), float(K), np.float32))


@pytest.mark.parametrize("tile_n", [128, 256, 512, 768])
def test_exact_small_integers_and_power_of_two_scales(tile_n):
    # codes in {0, +-1, +-2}, power-of-two scales: every partial sum is exact in FP32 in any order
    rng = np.random.default_rng(1)
    M, N, K = 256, 256, 1024
    nib = np.array([0, 2, 4, 10, 12], dtype=np.uint8)  # 0, 1, 2, -1, -2

    def make(R):
        c = nib[rng.integers(0, 5, size=(R, K))]
        codes = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
        scales = (rng.integers(5, 10, size=(R, K // 16)).astype(np.uint8) << 3)  # 2^-2 .. 2^2
        return oracle.Quantized(codes, scales, np.array([1.0, 0.5], np.float32), R, K)

    a, b = make(M), make(N)
    Dref, _ = P.gemm_reference(a, b)
    D = run_gemm(a, b, True, tile_n)
    assert np.array_equal(D.astype(np.float64), Dref)


@pytest.mark.parametrize("shape", [(128, 128, 256), (256, 384, 512), (384, 640, 768), (128, 256, 2048),
                                   (256, 256, 256), (512, 768, 1024), (256, 512, 3072)])
@pytest.mark.parametrize("tile_n", [128, 256, 512, 768])
@pytest.mark.parametrize("fp32", [False, True])
def test_against_fp64_product_of_decoded_operands(shape, tile_n, fp32):
    M, N, K = shape
    if tile_n == 512 and (M % 256 or N % 256):
        pytest.skip("CTA-pair tiles need M and N to be multiples of 256")
    a, b = operands(M, N, K, 40 + M + N)
    Dref, T = P.gemm_reference(a, b)
    D = run_gemm(a, b, fp32, tile_n)
    P.assert_gemm_close(D, Dref, T, not fp32, f"{shape} tile_n={tile_n}")


def test_many_tiles_per_cta_and_row_identity():
    # more tiles than SMs so that every CTA loops; operands with a distinct value per row / column block catch
    # any mix-up of tile coordinates or scale atoms
    M, N, K = 2048, 2560, 512
    a, b = operands(M, N, K, 9)
    a.scales[:] = np.clip(a.scales.astype(int) - (np.arange(M)[:, None] // 128 % 4) * 8, 1, 0x7E).astype(np.uint8)
    rows = np.arange(0, M, 37)
    cols = np.arange(0, N, 41)
    Dr, Tr = P.gemm_reference(a, b, rows=rows)
    Dc, Tc = P.gemm_reference(a, b, cols=cols)
    for tile_n in (256, 512):
        D = run_gemm(a, b, True, tile_n)
        P.assert_gemm_close(D[rows], Dr, Tr, False, f"sampled rows, tile_n={tile_n}")
        P.assert_gemm_close(D[:, cols], Dc, Tc, False, f"sampled cols, tile_n={tile_n}")


@pytest.mark.parametrize("tile_n", [128, 512])
def test_accumulate_into_fp32_and_leading_dimension(tile_n):
    M, N, K = 256, 256, 256
    a, b = operands(M, N, K, 3)
    Dref, T = P.gemm_reference(a, b)
    D0 = torch.randn((M, N), dtype=torch.float32, device="cuda")
    D = run_gemm(a, b, True, tile_n, accumulate=True, D0=D0)
    P.assert_gemm_close(D - D0.cpu().numpy(), Dref, T + np.abs(D0.cpu().numpy()) * 1e-3, False, "accumulate")
    # output embedded in a wider buffer: columns outside [0, N) stay untouched
    A, Bt = P.upload(a), P.upload(b)
    wide = torch.full((M, N + 64), 7.0, dtype=torch.bfloat16, device="cuda")
    B.nvfp4_set_gemm_tile_n(tile_n)
    try:
        B.nvfp4_gemm(A, Bt, wide[:, :N])
        B.nvfp4_device_status()
    finally:
        B.nvfp4_set_gemm_tile_n(0)
    assert torch.all(wide[:, N:] == 7.0)
    P.assert_gemm_close(wide[:, :N].float().cpu().numpy(), Dref, T, True, "ldd > N")


@pytest.mark.parametrize("tile_n", [256, 512])
def test_gemm_is_deterministic(tile_n):
    a, b = operands(256, 256, 1024, 5)
    D1, D2 = run_gemm(a, b, True, tile_n), run_gemm(a, b, True, tile_n)
    assert np.array_equal(D1, D2)


@pytest.mark.parametrize("shape", [(256, 384, 256), (256, 640, 512), (512, 768, 1024), (256, 1152, 768), (512, 512, 512),
                                   (768, 1408, 256), (256, 256, 2048)])
@pytest.mark.parametrize("fp32", [False, True])
def test_wide_tiles_against_fp64_product(shape, fp32):
    """256 x 384 tiles: N = 384 a + 256 b with every b in {0, 1, 2}, one and several k-blocks, both outputs."""
    M, N, K = shape
    a, b = operands(M, N, K, 41)
    Dref, T = P.gemm_reference(a, b)
    P.assert_gemm_close(run_gemm(a, b, fp32, 768), Dref, T, not fp32, f"wide {shape}")


def test_wide_tiles_exact_pairing_and_accumulate():
    rng = np.random.default_rng(9)
    M, N, K = 512, 1408, 1024  # three wide tiles + one narrow... 1408 = 11 x 128 = 384 * 1 + 256 * 4? no: q = 11 -> b = 1, a = 3
    nib = np.array([0, 2, 4, 10, 12], dtype=np.uint8)  # 0, 1, 2, -1, -2

    def make(R):
        c = nib[rng.integers(0, 5, size=(R, K))]
        codes = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
        scales = (rng.integers(5, 10, size=(R, K // 16)).astype(np.uint8) << 3)  # 2^-2 .. 2^2
        return oracle.Quantized(codes, scales, np.array([1.0, 0.5], np.float32), R, K)

    a, b = make(M), make(N)
    Dref, _ = P.gemm_reference(a, b)
    assert np.array_equal(run_gemm(a, b, True, 768).astype(np.float64), Dref)  # every partial sum exact
    D0 = torch.randn((M, N), device="cuda")
    D = run_gemm(a, b, True, 768, accumulate=True, D0=D0)
    assert np.allclose(D - D0.cpu().numpy(), Dref, rtol=0, atol=1e-3 * np.abs(D0.cpu().numpy()).max() + 1e-3)
