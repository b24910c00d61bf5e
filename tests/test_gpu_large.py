"""Edge of the size range: a tensor with more than 2^31 elements (element indices, code offsets and the 64-bit
stochastic-rounding counter must not wrap) and a GEMM with a thousand row blocks.  Inputs are drawn on the device in
chunks; the oracle remakes sampled slabs from the same bytes."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth
from test_gpu_fullsize import check_copy_slabs

pytestmark = pytest.mark.gpu


def _big_tensor(R, C, seed, std):
    x = torch.empty((R, C), dtype=torch.bfloat16, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(seed)
    for r0 in range(0, R, 8192):
        r1 = min(R, r0 + 8192)
        x[r0:r1] = (torch.randn((r1 - r0, C), generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)
    return x


def test_quantize_more_than_2_pow_31_elements():
    R, C = 69632, 32768  # 2.28e9 elements; element 2^31 is the first of row 65536
    assert R * C > 2 ** 31
    x = _big_tensor(R, C, 5, 1e-3)
    x[65536, 7] = 0.5  # the tensor amax sits just past the 2^31 boundary
    row, col = B.alloc_tensor(R, C), B.alloc_tensor(C, R)
    mask = synth.DEFAULT_RHT_SIGN_MASK
    B.nvfp4_quantize(x, B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=mask, seed=3,
                                     sr_offset=(1 << 40) + 9), row, col)
    torch.cuda.synchronize()
    assert float(row.glob[0]) == 0.5

    class Slabs:  # a source that only materialises the sampled row slabs on the host
        shape = (R, C)

        def __getitem__(self, sl):
            return x[sl].cpu()

    kw = dict(rounding=oracle.SR, seed=3, sr_offset=(1 << 40) + 9)
    # check_copy_slabs samples the first, an interior and the last slab; add the one that straddles 2^31
    check_copy_slabs(Slabs(), row, colwise=False, what="big row", **kw)
    check_copy_slabs(Slabs(), col, colwise=True, rht=True, mask=mask, what="big col", **kw)
    codes, scales, glob = P.download(row)
    r0 = 65536 - 64
    slab = synth.bits(x[r0:r0 + 128].cpu())
    ref = oracle.quantize(slab, amax_override=float(glob[0]), sr_row0=r0, sr_cols=C, **kw)
    assert np.array_equal(codes[r0:r0 + 128], ref.codes) and np.array_equal(scales[r0:r0 + 128], ref.scales)


def test_gemm_with_a_thousand_row_blocks():
    M, N, K = 131072, 512, 256
    a_src = _big_tensor(M, K, 6, 1.0)
    b_src = _big_tensor(N, K, 7, 0.02)
    A, Bt = B.alloc_tensor(M, K), B.alloc_tensor(N, K)
    B.nvfp4_quantize(a_src, B.quant_opts(), A, None)
    B.nvfp4_quantize(b_src, B.quant_opts(block_rows=16), Bt, None)
    D = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.nvfp4_gemm(A, Bt, D)
    B.nvfp4_device_status()
    assert torch.isfinite(D.float()).all()
    rows = np.array([0, 1, 255, 256, 65535, 65536, 100000, M - 257, M - 1])
    amax_a, amax_b = float(A.glob[0]), float(Bt.glob[0])
    b = oracle.quantize(synth.bits(b_src.cpu()), block_rows=16, amax_override=amax_b)
    for r in rows:
        g0 = (int(r) // 16) * 16
        a = oracle.quantize(synth.bits(a_src[g0:g0 + 16].cpu()), amax_override=amax_a)
        Dref, T = P.gemm_reference(a, b, rows=[int(r) - g0])
        P.assert_gemm_close(D[int(r)].float().cpu().numpy()[None, :], Dref, T, True, f"row {r}")


def test_bf16_gemm_with_more_than_2_pow_31_outputs_and_row_scaled_copy_past_the_boundary():
    """Variants at the edge of the size range: a BF16 GEMM whose output has 2.7e9 elements (exact integer data,
    sampled rows compared in full) and the one-pass row-scaled quantizer on a tensor with more than 2^31 elements
    (the draw counter and the code offsets of the last rows must not wrap)."""
    M, N, K = 65536, 40960, 64
    g = torch.Generator(device="cuda").manual_seed(7)
    a = torch.randint(-2, 3, (M, K), generator=g, device="cuda").to(torch.bfloat16)
    b = torch.randint(-2, 3, (N, K), generator=g, device="cuda").to(torch.bfloat16)
    D = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    assert D.numel() > 2 ** 31
    B.nvfp4_gemm_bf16(a, b, D)
    B.nvfp4_device_status()
    rows = torch.tensor([0, 255, 256, 32767, 52428, 52429, 65535], device="cuda")  # 52429 * 40960 > 2^31
    ref = oracle.gemm_tn(a[rows].float().cpu().numpy(), b.float().cpu().numpy(), want_T=False)
    assert np.array_equal(D[rows].float().cpu().numpy().astype(np.float64), ref)  # |sum| <= 256: exact in bf16
    del D

    R, C = 139264, 16384  # 2.28e9 elements, rows held by four warps
    x = _big_tensor(R, C, 9, 1.0)
    t = B.alloc_tensor(R, C, format=B.FORMAT_NVFP4_ROWSCALE)
    B.nvfp4_quantize(x, B.quant_opts(rounding=B.ROUND_STOCHASTIC, seed=4, sr_offset=(1 << 33) + 5), t, None)
    torch.cuda.synchronize()
    for r0 in (0, 131072, R - 128):  # 131072 * 16384 = 2^31
        ref = oracle.quantize_rowscale(synth.bits(x[r0:r0 + 128].cpu()), rounding=oracle.SR, seed=4,
                                       sr_offset=(1 << 33) + 5, sr_row0=r0, sr_cols=C)
        assert np.array_equal(t.codes[r0:r0 + 128].cpu().numpy(), ref.codes), f"codes of rows {r0}.."
        assert np.array_equal(t.glob.view(R, 2)[r0:r0 + 128].cpu().numpy().view(np.uint32), ref.glob.view(np.uint32))
        sc = t.scales.view(-1)[(r0 // 128) * (C // 64) * 512:((r0 // 128) + 1) * (C // 64) * 512].cpu().numpy()
        assert np.array_equal(oracle.sf_unswizzle(sc, 128, C // 16), ref.scales), f"scales of rows {r0}.."
