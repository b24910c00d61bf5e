"""Config 1 (single NVFP4 linear layer, fwd + bwd) through nvfp4_linear_fwd / nvfp4_linear_bwd vs the oracle."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def run_layer(p: synth.LinearProblem):
    M, N, K = p.M, p.N, p.K
    X, W, dY = p.X.cuda(), p.W.cuda(), p.dY.cuda()
    opts = B.quant_opts(rht_sign_mask=p.rht_sign_mask, seed=p.sr_seed, sr_offset=p.sr_offset)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    return Y, dX, dW, X_col, W_row, W_col


def test_config1_forward_and_backward_match_the_oracle():
    p = synth.config1()
    Y, dX, dW, X_col, W_row, W_col = run_layer(p)
    xb, wb, gb = synth.bits(p.X), synth.bits(p.W), synth.bits(p.dY)
    # saved operands
    P.assert_exact(W_row, oracle.quantize(wb, block_rows=16), "W row")
    P.assert_exact(W_col, oracle.quantize(wb, block_rows=16, colwise=True), "W col")
    # Fprop: Y = X_row W_row^T.  The GEMM is compared with the product of the operands the GPU itself produced
    # where those are only tolerance-equal to the oracle's (rotated copies), and with the oracle's otherwise.
    x_row = oracle.quantize(xb)
    w_row = oracle.quantize(wb, block_rows=16)
    Dref, T = P.gemm_reference(x_row, w_row)
    P.assert_gemm_close(Y.float().cpu().numpy(), Dref, T, True, "Fprop")
    # Dgrad: dX = dY_row W_col^T, dY quantized with stochastic rounding (bit-exact stream)
    g_row = oracle.quantize(gb, rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset)
    w_col = oracle.quantize(wb, block_rows=16, colwise=True)
    Dref, T = P.gemm_reference(g_row, w_col)
    P.assert_gemm_close(dX.float().cpu().numpy(), Dref, T, True, "Dgrad")
    # Wgrad: dW = dY_col X_col^T with both operands rotated.  X_col is an output of the forward call; dY_col lives in
    # the workspace and is reproduced by nvfp4_quantize with the same options (the kernels are deterministic).  Both
    # copies go through the tolerance protocol against the oracle first; then dW is held to the GEMM bound against
    # the FP64 product of those very operand bytes, decoded by the oracle, with no excused entries.
    y_col = B.nvfp4_rht16(p.X.cuda(), True, p.rht_sign_mask).cpu().numpy()
    P.assert_rht_close(xb, X_col, y_col, colwise=True, sign_mask=p.rht_sign_mask, rounding=oracle.RNE, what="X col")
    g_row_gpu, g_col_gpu = B.alloc_tensor(p.M, p.N), B.alloc_tensor(p.N, p.M)
    B.nvfp4_quantize(p.dY.cuda(), B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True,
                                               rht_sign_mask=p.rht_sign_mask, seed=p.sr_seed, sr_offset=p.sr_offset),
                     g_row_gpu, g_col_gpu)
    P.assert_exact(g_row_gpu, g_row, "dY row")
    g_y = B.nvfp4_rht16(p.dY.cuda(), True, p.rht_sign_mask).cpu().numpy()
    P.assert_rht_close(gb, g_col_gpu, g_y, colwise=True, sign_mask=p.rht_sign_mask, rounding=oracle.SR,
                       seed=p.sr_seed, sr_offset=p.sr_offset, what="dY col")
    Dref, T = oracle.gemm_tn(P.decode_rows(g_col_gpu, np.arange(p.N)), P.decode_rows(X_col, np.arange(p.K)))
    dWn = dW.cpu().numpy()
    P.assert_gemm_close(dWn, Dref, T, False, "Wgrad")
    # and the whole layer approximates the unquantized gradients
    exact = p.dY.double().numpy().T @ p.X.double().numpy()
    assert np.linalg.norm(dWn - exact) / np.linalg.norm(exact) < 0.25


def test_cached_weight_and_skipped_outputs():
    p = synth.config1()
    Y, dX, dW, X_col, W_row, W_col = run_layer(p)
    M, N, K = p.M, p.N, p.K
    opts = B.quant_opts(rht_sign_mask=p.rht_sign_mask, seed=p.sr_seed, sr_offset=p.sr_offset)
    Y2 = torch.empty_like(Y)
    ws = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    B.nvfp4_linear_fwd(p.X.cuda(), None, opts, Y2, None, W_row, None, True, ws)
    assert torch.equal(Y, Y2)
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    dX2 = torch.empty_like(dX)
    B.nvfp4_linear_bwd(p.dY.cuda(), None, W_col, K, opts, dX2, None, False, ws_b)
    assert torch.equal(dX, dX2)
    dW2 = dW.clone()
    B.nvfp4_linear_bwd(p.dY.cuda(), X_col, None, K, opts, None, dW2, True, ws_b)
    B.nvfp4_device_status()
    assert torch.allclose(dW2, 2 * dW, rtol=1e-6, atol=0)


@pytest.mark.parametrize("M,N,K,with_col", [
    (256, 5120, 1024, True),    # W has far more tiles than X: most CTAs only carry tiles of W
    (4096, 256, 512, True),     # the reverse: few tiles of W among many of X
    (1024, 2304, 768, False),   # forward only (no transposed copies): the row-wise variant of the kernel
    (8192, 6144, 2560, True),   # more tiles of both than resident CTAs: every CTA interleaves the two kinds
])
def test_forward_call_quantizes_w_exactly_like_the_standalone_call(M, N, K, with_col):
    """The forward call takes W's tensor amax (Appendix B.1) inside the kernel that quantizes X; the standalone call
    runs its own amax pass.  Every byte of the W and X copies, the global scales and Y must agree."""
    g = torch.Generator(device="cuda").manual_seed(M + N + K)
    X = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    # the tensor amax sits in one corner tile each time (first, last, and a middle tile)
    for pos in ((0, 0), (N - 1, K - 1), (N // 2 + 3, K // 2 + 5)):
        Wp = W.clone()
        Wp[pos] = -3.0
        opts = B.quant_opts(rht_sign_mask=synth.DEFAULT_RHT_SIGN_MASK)
        X_col = B.alloc_tensor(K, M) if with_col else None
        W_row, W_col = B.alloc_tensor(N, K), (B.alloc_tensor(K, N) if with_col else None)
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
        B.nvfp4_linear_fwd(X, Wp, opts, Y, X_col, W_row, W_col, False, ws)
        W_row2, W_col2 = B.alloc_tensor(N, K), (B.alloc_tensor(K, N) if with_col else None)
        B.nvfp4_quantize(Wp, B.quant_opts(block_rows=16), W_row2, W_col2)
        X_row2, X_col2 = B.alloc_tensor(M, K), (B.alloc_tensor(K, M) if with_col else None)
        B.nvfp4_quantize(X, B.quant_opts(rht_colwise=True, rht_sign_mask=synth.DEFAULT_RHT_SIGN_MASK), X_row2, X_col2)
        Y2 = torch.empty_like(Y)
        B.nvfp4_gemm(X_row2, W_row2, Y2)
        B.nvfp4_device_status()
        pairs = [(W_row, W_row2)] + ([(W_col, W_col2), (X_col, X_col2)] if with_col else [])
        for a, b in pairs:
            assert torch.equal(a.codes, b.codes) and torch.equal(a.scales, b.scales)
            assert torch.equal(a.glob, b.glob)
        assert float(W_row.glob[0]) == 3.0
        assert torch.equal(Y, Y2)
