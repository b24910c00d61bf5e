"""Parity at the remaining benchmark shapes, in the launch configuration `bench.py --config 4|5` times:
cfg 4 (FFN down-projection, M 8192, K 20480, N 5120, squared-ReLU input) forward AND backward, and the out-projection,
FFN-up and FFN-down layers of cfg 5 at 16384 tokens, all through nvfp4_linear_fwd / nvfp4_linear_bwd.
The tensors are drawn on the device; the oracle remakes sampled slabs of every operand copy and sampled rows x
columns of every GEMM from slabs read back from the device."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth
from test_gpu_fullsize import Operand, check_copy_slabs, check_gemm_samples

pytestmark = pytest.mark.gpu


def rotated_amax_device(x: torch.Tensor, mask: int) -> float:
    """max |x^T (S H_16)| with 16-chunks down the rows, in float64 on the device (a torch matmul, not the kernels)."""
    H = torch.tensor([[oracle.hadamard16_entry(j, k) for k in range(16)] for j in range(16)], dtype=torch.float64)
    s = torch.tensor([-1.0 if (mask >> j) & 1 else 1.0 for j in range(16)], dtype=torch.float64)
    SH = ((s[:, None] * H) / 4).to(x.device)
    best = 0.0
    for r0 in range(0, x.shape[0], 512):
        blk = x[r0:r0 + 512].to(torch.float64).reshape(-1, 16, x.shape[1])
        best = max(best, float(torch.einsum("qjc,jk->qkc", blk, SH).abs().max()))
    return best


def run_and_check_layer(p: synth.LinearProblem, seed: int):
    M, N, K, mask = p.M, p.N, p.K, p.rht_sign_mask
    X, W, dY = p.X, p.W, p.dY  # device tensors
    opts = B.quant_opts(rht_sign_mask=mask, seed=p.sr_seed, sr_offset=p.sr_offset)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
    B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    del ws_f, ws_b
    # the copies the two calls keep in their workspaces, reproduced with the same options (deterministic kernels)
    X_row, X_col2 = B.alloc_tensor(M, K), B.alloc_tensor(K, M)
    B.nvfp4_quantize(X, B.quant_opts(rht_colwise=True, rht_sign_mask=mask), X_row, X_col2)
    g_row, g_col = B.alloc_tensor(M, N), B.alloc_tensor(N, M)
    sr_opts = B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=mask, seed=p.sr_seed,
                           sr_offset=p.sr_offset)
    B.nvfp4_quantize(dY, sr_opts, g_row, g_col)
    torch.cuda.synchronize()
    assert torch.equal(X_col2.codes, X_col.codes) and torch.equal(X_col2.scales, X_col.scales)
    del X_col2

    # tensor amax: plain ones exactly, rotated ones within 1e-5 of a float64 evaluation
    assert float(X_row.glob[0]) == float(X.abs().max().float())
    assert float(W_row.glob[0]) == float(W.abs().max().float()) == float(W_col.glob[0])
    assert float(g_row.glob[0]) == float(dY.abs().max().float())
    for t, src in ((X_col, X), (g_col, dY)):
        ref = rotated_amax_device(src, mask)
        assert abs(float(t.glob[0]) - ref) <= 1e-5 * ref

    sr = dict(rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset)
    check_copy_slabs(X, X_row, colwise=False, what=f"{p.name} X row")
    check_copy_slabs(X, X_col, colwise=True, rht=True, mask=mask, what=f"{p.name} X col")
    check_copy_slabs(W, W_row, colwise=False, block_rows=16, what=f"{p.name} W row")
    check_copy_slabs(W, W_col, colwise=True, block_rows=16, what=f"{p.name} W col")
    check_copy_slabs(dY, g_row, colwise=False, what=f"{p.name} dY row", **sr)
    check_copy_slabs(dY, g_col, colwise=True, rht=True, mask=mask, what=f"{p.name} dY col", **sr)

    o_x_row, o_x_col = Operand(X_row, X, colwise=False), Operand(X_col, X, colwise=True, rht=True, mask=mask)
    o_w_row, o_w_col = Operand(W_row, W, colwise=False, block_rows=16), Operand(W_col, W, colwise=True, block_rows=16)
    o_g_row, o_g_col = Operand(g_row, dY, colwise=False, **sr), Operand(g_col, dY, colwise=True, rht=True, mask=mask, **sr)
    check_gemm_samples(Y, o_x_row, o_w_row, True, f"{p.name} Fprop", seed)
    check_gemm_samples(dX, o_g_row, o_w_col, True, f"{p.name} Dgrad", seed + 1)
    check_gemm_samples(dW, o_g_col, o_x_col, False, f"{p.name} Wgrad", seed + 2)
    for t in (Y, dX, dW):
        assert torch.isfinite(t.float()).all()
    # the quantized layer approximates the unquantized products (a property that holds at any size)
    rows = torch.arange(0, M, 1999, device="cuda")
    exact = X[rows].double() @ W.double().T
    assert float((Y[rows].double() - exact).norm() / exact.norm()) < 0.2
    cols = torch.arange(0, N, 257, device="cuda")
    exact = dY[:, cols].double().T @ X.double()
    assert float((dW[cols].double() - exact).norm() / exact.norm()) < 0.3


def test_config4_full_size_forward_and_backward():
    """K = 20480: the Wgrad operand X_col has 20480 rows rotated along 8192 tokens; half of X is exactly zero."""
    p = synth.config4_device()
    assert float((p.X == 0).float().mean()) > 0.4
    run_and_check_layer(p, 40)


@pytest.mark.parametrize("layer", [1, 2, 3])
def test_config5_layers_at_16384_tokens(layer):
    """Out-projection (5120 x 5120), FFN up (20480 x 5120) and FFN down (5120 x 20480, squared-ReLU input) at 16384
    tokens: Wgrad contracts over 16384 tokens, the FFN-down input has 335 M elements."""
    run_and_check_layer(synth.config5_layer_device(layer), 50 + 10 * layer)
