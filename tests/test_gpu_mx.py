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


@pytest.mark.parametrize("shape", [(128, 128, 256), (384, 640, 768), (256, 256, 1024)])
@pytest.mark.parametrize("tile_n", [128, 256])
@pytest.mark.parametrize("fp32", [False, True])
def test_gemm_one_cta_kernel(shape, tile_n, fp32):
    """Shapes with M or N not a multiple of 256 (and the forced tile widths) take the one-CTA kernel."""
    M, N, K = shape
    a = oracle.quantize_mx(synth.bits(synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, 35, 36)))
    b = oracle.quantize_mx(synth.bits(synth.normal_bf16((N, K), 0.02, 37)), block_rows=32)
    Dref, T = reference(a, b)
    B.nvfp4_set_gemm_tile_n(tile_n)
    try:
        D = run_gemm(a, b, fp32)
    finally:
        B.nvfp4_set_gemm_tile_n(0)
    P.assert_gemm_close(D, Dref, T, not fp32, f"mx one-CTA {shape} tile {tile_n}")
    if shape == (256, 256, 1024) and fp32:  # exact pairing of scale bytes with blocks in this kernel too
        rng = np.random.default_rng(6)
        mk = lambda R: oracle.QuantizedMX(np.full((R, K // 2), 0x22, np.uint8),
                                          (127 + rng.integers(-3, 4, size=(R, K // 32))).astype(np.uint8), R, K)
        a, b = mk(M), mk(N)
        B.nvfp4_set_gemm_tile_n(tile_n)
        try:
            D = run_gemm(a, b, True)
        finally:
            B.nvfp4_set_gemm_tile_n(0)
        assert np.array_equal(D.astype(np.float64), reference(a, b)[0])


def test_gemm_rejects_mixed_formats():
    n = P.upload(oracle.quantize(synth.bits(synth.normal_bf16((256, 256), 1.0, 2))))
    m = upload_mx(oracle.quantize_mx(synth.bits(synth.normal_bf16((256, 256), 1.0, 3))))
    with pytest.raises(B.NVFP4Error) as e:
        B.nvfp4_gemm(n, m, torch.empty((256, 256), dtype=torch.float32, device="cuda"))
    assert e.value.status == 4


# ------------------------------------------------------------------------------- quantizer ----
MASK32 = 0xA5C373E5


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (512, 1024), (32, 32), (160, 224), (96, 416)])
@pytest.mark.parametrize("which", ["row", "col", "both"])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_quantize_1x32_is_bit_exact(shape, which, rounding):
    x = synth.normal_with_outliers_bf16(shape, 0.01, 50.0, 41, 42)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    row, col = P.gpu_quantize_mx(x, rowwise=which != "col", colwise=which != "row", sf_layout=layout,
                                 rounding=rounding, seed=7, sr_offset=3)
    kw = dict(rounding=rounding, seed=7, sr_offset=3)
    if row is not None:
        P.assert_exact_mx(row, oracle.quantize_mx(synth.bits(x), **kw), f"row {shape}")
    if col is not None:
        P.assert_exact_mx(col, oracle.quantize_mx(synth.bits(x), colwise=True, **kw), f"col {shape}")


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (160, 224)])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_quantize_32x32_weights_bit_exact_and_consistent(shape, rounding):
    w = synth.normal_bf16(shape, 0.02, 43)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    row, col = P.gpu_quantize_mx(w, colwise=True, sf_layout=layout, block_rows=32, rounding=rounding, seed=1)
    kw = dict(block_rows=32, rounding=rounding, seed=1)
    P.assert_exact_mx(row, oracle.quantize_mx(synth.bits(w), **kw), "2d row")
    P.assert_exact_mx(col, oracle.quantize_mx(synth.bits(w), colwise=True, **kw), "2d col")
    if rounding == B.ROUND_NEAREST_EVEN:
        rc, _ = P.download_mx(row)
        cc, _ = P.download_mx(col)
        assert np.array_equal(P.unpack(rc), P.unpack(cc).T), "the transposed copy holds the same codes"


@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (160, 224)])
@pytest.mark.parametrize("rounding", [B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC])
def test_quantize_rht32_copy_follows_the_tolerance_protocol(shape, rounding):
    x = synth.normal_with_outliers_bf16(shape, 0.01, 50.0, 45, 46)
    layout = B.SF_SWIZZLED if shape[0] % 128 == 0 and shape[1] % 128 == 0 else B.SF_LINEAR
    row, col = P.gpu_quantize_mx(x, colwise=True, sf_layout=layout, rounding=rounding, rht_colwise=True,
                                 rht_sign_mask=MASK32, seed=2, sr_offset=5)
    P.assert_exact_mx(row, oracle.quantize_mx(synth.bits(x), rounding=rounding, seed=2, sr_offset=5), "row beside rht col")
    st = P.assert_mx_rht_close(synth.bits(x), col, colwise=True, sign_mask=MASK32, rounding=rounding, seed=2,
                               sr_offset=5, what=f"rht col {shape}")
    assert st["excused_codes"] + st["excused_scales"] <= max(1e-3 * st["elements"], 32)


def test_quantize_degenerate_and_rejected_inputs():
    z = torch.zeros((128, 128), dtype=torch.bfloat16)
    row, col = P.gpu_quantize_mx(z, colwise=True)
    P.assert_exact_mx(row, oracle.quantize_mx(synth.bits(z)), "zeros row")
    P.assert_exact_mx(col, oracle.quantize_mx(synth.bits(z), colwise=True), "zeros col")
    for scale in (1e-36, 3e-39, 1e30):
        x = (synth.normal_bf16((128, 128), 1.0, 21).float() * scale).to(torch.bfloat16)
        row, col = P.gpu_quantize_mx(x, colwise=True)
        P.assert_exact_mx(row, oracle.quantize_mx(synth.bits(x)), f"row scale {scale}")
        P.assert_exact_mx(col, oracle.quantize_mx(synth.bits(x), colwise=True), f"col scale {scale}")
    x = synth.normal_bf16((48, 64), 1.0, 1).cuda()  # 48 rows: not a multiple of 32
    with pytest.raises(B.NVFP4Error) as e:
        B.nvfp4_quantize(x, B.quant_opts(), B.alloc_tensor(48, 64, B.SF_LINEAR, format=B.FORMAT_MXFP4), None)
    assert e.value.status == 2
    x = synth.normal_bf16((64, 64), 1.0, 1).cuda()
    with pytest.raises(B.NVFP4Error) as e:  # 16x16 blocks belong to the other format
        B.nvfp4_quantize(x, B.quant_opts(block_rows=16), B.alloc_tensor(64, 64, B.SF_LINEAR, format=B.FORMAT_MXFP4), None)
    assert e.value.status == 4
    with pytest.raises(B.NVFP4Error) as e:  # the two copies must share a format
        B.nvfp4_quantize(x, B.quant_opts(), B.alloc_tensor(64, 64, B.SF_LINEAR, format=B.FORMAT_MXFP4),
                         B.alloc_tensor(64, 64, B.SF_LINEAR))
    assert e.value.status == 4


def test_quantize_then_gemm_matches_the_oracle_pipeline():
    """Wgrad-like use: both operands transposed copies with the 32-point transform, gradients stochastically rounded."""
    M, N, K = 512, 256, 256  # tokens, out features, in features
    X = synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, 51, 52)
    dY = synth.normal_bf16((M, N), 1e-3, 53)
    _, x_col = P.gpu_quantize_mx(X, rowwise=False, colwise=True, rht_colwise=True, rht_sign_mask=MASK32)
    _, g_col = P.gpu_quantize_mx(dY, rowwise=False, colwise=True, rht_colwise=True, rht_sign_mask=MASK32,
                                 rounding=B.ROUND_STOCHASTIC, seed=4)
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    B.nvfp4_gemm(g_col, x_col, dW)
    B.nvfp4_device_status()
    # reference: the oracle's own pipeline; the few codes the tolerance protocol may excuse move single products
    x_ref = oracle.quantize_mx(synth.bits(X), colwise=True, rht=True, sign_mask=MASK32)
    g_ref = oracle.quantize_mx(synth.bits(dY), colwise=True, rht=True, sign_mask=MASK32, rounding=oracle.SR, seed=4)
    Dref, T = oracle.gemm_tn(oracle.dequantize_mx(g_ref), oracle.dequantize_mx(x_ref))
    err = np.abs(dW.cpu().numpy() - Dref)
    assert np.count_nonzero(err > 1e-3 * T) <= 1e-3 * err.size
    assert np.all(err <= 2e-2 * T)
    exact = dY.double().numpy().T @ X.double().numpy()
    assert np.linalg.norm(dW.cpu().numpy() - exact) / np.linalg.norm(exact) < 0.35  # the transform cancels


def test_linear_layer_in_mxfp4_matches_the_oracle_pipeline():
    """fwd + bwd of one layer with MXFP4 copies: every stored operand against the oracle, the three products against
    the FP64 product of the oracle's own operands."""
    M, N, K = 512, 768, 256
    X = synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, 61, 62)
    W = synth.normal_bf16((N, K), 0.02, 63)
    dY = synth.normal_bf16((M, N), 1e-3, 64)
    mx = dict(format=B.FORMAT_MXFP4)
    X_col, W_row, W_col = B.alloc_tensor(K, M, **mx), B.alloc_tensor(N, K, **mx), B.alloc_tensor(K, N, **mx)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    opts = B.quant_opts(rht_sign_mask=MASK32, seed=9, sr_offset=1)
    B.nvfp4_linear_fwd(X.cuda(), W.cuda(), opts, Y, X_col, W_row, W_col, False, ws_f)
    B.nvfp4_linear_bwd(dY.cuda(), X_col, W_col, K, opts, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    xb, wb, gb = synth.bits(X), synth.bits(W), synth.bits(dY)
    w_row, w_col = oracle.quantize_mx(wb, block_rows=32), oracle.quantize_mx(wb, block_rows=32, colwise=True)
    P.assert_exact_mx(W_row, w_row, "W row")
    P.assert_exact_mx(W_col, w_col, "W col")
    P.assert_mx_rht_close(xb, X_col, colwise=True, sign_mask=MASK32, rounding=oracle.RNE, what="X col")
    deq = oracle.dequantize_mx
    Dref, T = oracle.gemm_tn(deq(oracle.quantize_mx(xb)), deq(w_row))
    P.assert_gemm_close(Y.float().cpu().numpy(), Dref, T, True, "Fprop")
    g_row = oracle.quantize_mx(gb, rounding=oracle.SR, seed=9, sr_offset=1)
    Dref, T = oracle.gemm_tn(deq(g_row), deq(w_col))
    P.assert_gemm_close(dX.float().cpu().numpy(), Dref, T, True, "Dgrad")
    g_col = oracle.quantize_mx(gb, colwise=True, rht=True, sign_mask=MASK32, rounding=oracle.SR, seed=9, sr_offset=1)
    x_col = oracle.quantize_mx(xb, colwise=True, rht=True, sign_mask=MASK32)
    Dref, T = oracle.gemm_tn(deq(g_col), deq(x_col))
    err = np.abs(dW.cpu().numpy() - Dref)
    assert np.count_nonzero(err > 1e-3 * T) <= 1e-3 * err.size and np.all(err <= 2e-2 * T)
    exact = dY.double().numpy().T @ X.double().numpy()
    assert np.linalg.norm(dW.cpu().numpy() - exact) / np.linalg.norm(exact) < 0.35
    # a layer cannot mix formats
    with pytest.raises(B.NVFP4Error) as e:
        B.nvfp4_linear_fwd(X.cuda(), W.cuda(), opts, Y, B.alloc_tensor(K, M), W_row, W_col, False, ws_f)
    assert e.value.status == 4


def test_full_size_layer_in_mxfp4_sampled():
    """The bench's cfg 3 layer (M 8192, K 5120, N 20480) in MXFP4: stored operands on sampled slabs, the three
    products on sampled rows x columns against operand rows the oracle remakes from the sources."""
    p = synth.config3()
    M, N, K = p.M, p.N, p.K
    mx = dict(format=B.FORMAT_MXFP4)
    X, W, dY = p.X.cuda(), p.W.cuda(), p.dY.cuda()
    X_col, W_row, W_col = B.alloc_tensor(K, M, **mx), B.alloc_tensor(N, K, **mx), B.alloc_tensor(K, N, **mx)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    opts = B.quant_opts(rht_sign_mask=MASK32, seed=p.sr_seed, sr_offset=p.sr_offset)
    B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
    B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    for t in (Y, dX, dW):
        assert torch.isfinite(t.float()).all()

    xb, wb, gb = synth.bits(p.X), synth.bits(p.W), synth.bits(p.dY)
    sr = dict(rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset)

    def rows_of(src_bits, rows, *, colwise, block_rows=1, rht=False, **kw):
        """Rows of a copy, remade by the oracle from 32-row (or 32-column) slabs of the source."""
        n_src_cols = src_bits.shape[1]
        codes, scales = [], []
        for r in rows:
            g0 = (int(r) // 32) * 32
            if colwise:
                q = oracle.quantize_mx(src_bits[:, g0:g0 + 32], colwise=True, block_rows=block_rows, rht=rht,
                                       sign_mask=MASK32, sr_cols=n_src_cols, sr_col0=g0, **kw)
            else:
                q = oracle.quantize_mx(src_bits[g0:g0 + 32], block_rows=block_rows, sr_cols=n_src_cols, sr_row0=g0, **kw)
            codes.append(q.codes[int(r) - g0])
            scales.append(q.scales[int(r) - g0])
        n_cols = src_bits.shape[0] if colwise else n_src_cols
        return oracle.QuantizedMX(np.stack(codes), np.stack(scales), len(rows), n_cols)

    # stored weight copies: sampled rows, bit-exact
    rng = np.random.default_rng(11)
    wr, wc = P.download_mx(W_row), P.download_mx(W_col)
    rows = np.sort(rng.choice(N, 8, replace=False))
    ref = rows_of(wb, rows, colwise=False, block_rows=32)
    assert np.array_equal(wr[0][rows], ref.codes) and np.array_equal(wr[1][rows], ref.scales)
    cols = np.sort(rng.choice(K, 8, replace=False))
    ref = rows_of(wb, cols, colwise=True, block_rows=32)
    assert np.array_equal(wc[0][cols], ref.codes) and np.array_equal(wc[1][cols], ref.scales)

    def check(D, a, b, rows, cols, bf16, loose, what):
        Dref, T = oracle.gemm_tn(oracle.dequantize_mx(a), oracle.dequantize_mx(b))
        got = D[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy()
        if loose:  # transformed operands: the few codes the protocol may excuse move single products
            err = np.abs(got - Dref)
            assert np.count_nonzero(err > 1e-3 * T + 1e-30) <= 1e-3 * err.size and np.all(err <= 2e-2 * T + 1e-30), what
        else:
            P.assert_gemm_close(got, Dref, T, bf16, what)

    r12 = np.sort(rng.choice(M, 12, replace=False))
    c256 = np.sort(rng.choice(N, 256, replace=False))
    check(Y, rows_of(xb, r12, colwise=False), rows_of(wb, c256, colwise=False, block_rows=32), r12, c256, True, False, "Fprop")
    k256 = np.sort(rng.choice(K, 256, replace=False))
    check(dX, rows_of(gb, r12, colwise=False, **sr), rows_of(wb, k256, colwise=True, block_rows=32), r12, k256, True, False,
          "Dgrad")
    n12 = np.sort(rng.choice(N, 12, replace=False))
    check(dW, rows_of(gb, n12, colwise=True, rht=True, **sr), rows_of(xb, k256, colwise=True, rht=True), n12, k256, False,
          True, "Wgrad")
