"""Parity at the benchmark's full size (cfg 3: M 8192, K 5120, N 20480) in the launch configuration bench.py times:
nvfp4_linear_fwd / nvfp4_linear_bwd for the GEMM outputs, nvfp4_quantize with the same options for the operand
copies.  The oracle checks sampled row slabs of every quantized copy and sampled rows / columns of every GEMM."""
import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def rotated_amax(x: torch.Tensor, mask: int) -> float:
    """max |x^T (S H_16)| over the whole tensor, chunks of 16 along the rows (tokens), in float64 (torch matmul)."""
    H = torch.tensor([[oracle.hadamard16_entry(j, k) for k in range(16)] for j in range(16)], dtype=torch.float64)
    s = torch.tensor([-1.0 if (mask >> j) & 1 else 1.0 for j in range(16)], dtype=torch.float64)
    SH = (s[:, None] * H) / 4
    best = 0.0
    for r0 in range(0, x.shape[0], 1024):
        blk = x[r0:r0 + 1024].to(torch.float64).reshape(-1, 16, x.shape[1])       # [chunks, 16, cols]
        y = torch.einsum("qjc,jk->qkc", blk, SH)
        best = max(best, float(y.abs().max()))
    return best


def check_copy_slabs(x: torch.Tensor, gpu: B.NVFP4Tensor, *, colwise, block_rows=1, rht=False, mask=0, rounding=0,
                     seed=0, sr_offset=0, what="", rht_dim=16):
    """Three 128-row slabs of the source (first, interior, last) remade by the oracle with the GPU's tensor amax:
    bit-exact for untransformed copies, the full tolerance protocol (threshold proximity of every differing scale
    byte and code, adjacency, at most 1e-3 of the elements) for transformed ones."""
    codes, scales, glob = P.download(gpu)
    R, n_cols = x.shape[0], x.shape[1]
    n_bad = n_tot = 0
    for r0 in (0, (R // 128) * 5 // 8 * 128 + 0, R - 128):
        slab = synth.bits(x[r0:r0 + 128].cpu())  # x may live on the device: only the slab comes to the host
        ref = oracle.quantize(slab, colwise=colwise, block_rows=block_rows, rht=rht, sign_mask=mask, rounding=rounding,
                              seed=seed, sr_offset=sr_offset, amax_override=float(glob[0]), sr_row0=r0,
                              sr_cols=n_cols, rht_dim=rht_dim, return_y=rht)
        assert glob.view(np.uint32)[1] == ref.glob.view(np.uint32)[1], f"{what}: s_dec"
        if colwise:
            got_c, got_s = codes[:, r0 // 2:(r0 + 128) // 2], scales[:, r0 // 16:(r0 + 128) // 16]
        else:
            got_c, got_s = codes[r0:r0 + 128], scales[r0:r0 + 128]
        if not rht:
            assert np.array_equal(got_s, ref.scales), f"{what}: scale bytes of slab {r0}"
            assert np.array_equal(got_c, ref.codes), f"{what}: codes of slab {r0}"
        else:
            # element (r, c) of the slab's copy is source element (r0 + c, r) for a transposed copy, (r0 + r, c) else
            draw = (lambda r, c: oracle.sr_draw(seed, sr_offset, (r0 + c) * n_cols + r)) if colwise else \
                   (lambda r, c: oracle.sr_draw(seed, sr_offset, (r0 + r) * n_cols + c))
            cnt = P.compare_rotated(got_c, got_s, ref, float(glob[0]), rounding, draw, f"{what}, slab {r0}")
            n_bad += cnt["excused_codes"] + 16 * cnt["excused_scales"]
        n_tot += got_c.size * 2
    assert n_bad <= 1e-3 * n_tot, f"{what}: {n_bad} of {n_tot} elements differ"


class Operand:
    """How an operand copy was made from its source, so that the oracle can remake any of its rows."""

    def __init__(self, gpu: B.NVFP4Tensor, src: torch.Tensor, *, colwise, block_rows=1, rht=False, mask=0, rounding=0,
                 seed=0, sr_offset=0):
        self.gpu, self.src = gpu, src
        self.kw = dict(colwise=colwise, block_rows=block_rows, rht=rht, sign_mask=mask, rounding=rounding, seed=seed,
                       sr_offset=sr_offset)
        self.colwise = colwise

    def oracle_rows(self, rows):
        """The sampled rows of the copy, quantized by the oracle from the source (groups of 16 rows of the copy;
        the tensor amax is the GPU's, as the comparison protocol prescribes)."""
        amax = float(self.gpu.glob[0])
        n_cols = self.gpu.cols
        codes = np.zeros((len(rows), n_cols // 2), np.uint8)
        scales = np.zeros((len(rows), n_cols // 16), np.uint8)
        glob = None
        for i, r in enumerate(rows):
            g0 = (int(r) // 16) * 16
            if self.colwise:  # only the 16 source columns / rows of the group are brought to the host
                q = oracle.quantize(synth.bits(self.src[:, g0:g0 + 16].cpu()), amax_override=amax,
                                    sr_cols=self.src.shape[1], sr_col0=g0, **self.kw)
            else:
                q = oracle.quantize(synth.bits(self.src[g0:g0 + 16].cpu()), amax_override=amax,
                                    sr_cols=self.src.shape[1], sr_row0=g0, **self.kw)
            codes[i], scales[i], glob = q.codes[int(r) - g0], q.scales[int(r) - g0], q.glob
        return oracle.Quantized(codes, scales, glob, len(rows), n_cols)


def check_gemm_samples(D: torch.Tensor, A: Operand, Bt: Operand, bf16: bool, what: str, seed: int):
    """Sampled rows x columns of a full-size product against the FP64 product of the decoded operands, held to
    1e-3 * sum|a||b| (+ the output rounding for bf16) with no exceptions.  Untransformed operand rows are remade by
    the ORACLE from the sources (their copies are bit-exact); for a transformed operand, whose copy may differ from
    the oracle's in the codes the protocol excuses, the rows are the device copy's own bytes (checked against the
    oracle by check_copy_slabs) decoded by the oracle: the GEMM is judged on the operands it was given."""
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(A.gpu.rows, 12, replace=False))
    cols = np.sort(rng.choice(Bt.gpu.rows, 384, replace=False))
    a = P.decode_rows(A.gpu, rows) if A.kw["rht"] else oracle.dequantize(A.oracle_rows(rows))
    b = P.decode_rows(Bt.gpu, cols) if Bt.kw["rht"] else oracle.dequantize(Bt.oracle_rows(cols))
    Dref, T = oracle.gemm_tn(a, b)
    got = D[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy()
    P.assert_gemm_close(got, Dref, T, bf16, what)


def test_config3_full_size_forward_and_backward():
    p = synth.config3()
    M, N, K = p.M, p.N, p.K
    mask = p.rht_sign_mask
    X, W, dY = p.X.cuda(), p.W.cuda(), p.dY.cuda()
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

    # the operand copies the two calls keep in their workspaces, reproduced with the same options
    X_row = B.alloc_tensor(M, K)
    X_col2 = B.alloc_tensor(K, M)
    B.nvfp4_quantize(X, B.quant_opts(rht_colwise=True, rht_sign_mask=mask), X_row, X_col2)
    g_row, g_col = B.alloc_tensor(M, N), B.alloc_tensor(N, M)
    B.nvfp4_quantize(dY, B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=mask,
                                      seed=p.sr_seed, sr_offset=p.sr_offset), g_row, g_col)
    torch.cuda.synchronize()
    assert torch.equal(X_col2.codes, X_col.codes) and torch.equal(X_col2.scales, X_col.scales)  # deterministic

    # ---- quantizer: tensor amax against torch, sampled slabs against the oracle -------------------------------
    assert float(X_row.glob[0]) == float(p.X.abs().max().float())
    assert float(W_row.glob[0]) == float(p.W.abs().max().float()) == float(W_col.glob[0])
    assert float(g_row.glob[0]) == float(p.dY.abs().max().float())
    for t, src in ((X_col, p.X), (g_col, p.dY)):
        ref = rotated_amax(src, mask)
        assert abs(float(t.glob[0]) - ref) <= 1e-5 * ref
    check_copy_slabs(p.X, X_row, colwise=False, what="X row")
    check_copy_slabs(p.X, X_col, colwise=True, rht=True, mask=mask, what="X col")
    check_copy_slabs(p.W, W_row, colwise=False, block_rows=16, what="W row")
    check_copy_slabs(p.W, W_col, colwise=True, block_rows=16, what="W col")
    check_copy_slabs(p.dY, g_row, colwise=False, rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset, what="dY row")
    check_copy_slabs(p.dY, g_col, colwise=True, rht=True, mask=mask, rounding=oracle.SR, seed=p.sr_seed,
                     sr_offset=p.sr_offset, what="dY col")

    # ---- GEMMs: sampled rows x columns against the FP64 product of the decoded operands -----------------------
    sr = dict(rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset)
    o_x_row, o_x_col = Operand(X_row, p.X, colwise=False), Operand(X_col, p.X, colwise=True, rht=True, mask=mask)
    o_w_row = Operand(W_row, p.W, colwise=False, block_rows=16)
    o_w_col = Operand(W_col, p.W, colwise=True, block_rows=16)
    o_g_row, o_g_col = Operand(g_row, p.dY, colwise=False, **sr), Operand(g_col, p.dY, colwise=True, rht=True, mask=mask, **sr)
    check_gemm_samples(Y, o_x_row, o_w_row, True, "Fprop", 1)
    check_gemm_samples(dX, o_g_row, o_w_col, True, "Dgrad", 2)
    check_gemm_samples(dW, o_g_col, o_x_col, False, "Wgrad", 3)
    # properties that hold at any size: no NaN / Inf, and the layer approximates the unquantized products
    for t in (Y, dX, dW):
        assert torch.isfinite(t.float()).all()
    rows = torch.arange(0, M, 997, device="cuda")
    exact = X[rows].double() @ W.double().T
    rel = float((Y[rows].double() - exact).norm() / exact.norm())
    assert rel < 0.2, rel


def test_config2_quantizer_sweep_full_tensor():
    """cfg 2: the [8192 x 5120] activation.  One full-tensor bit-exact comparison (RNE, both copies, no transform);
    the SR and rotated variants on sampled slabs."""
    x = synth.config2_x()
    xd = x.cuda()
    R, C = x.shape
    row, col = B.alloc_tensor(R, C), B.alloc_tensor(C, R)
    B.nvfp4_quantize(xd, B.quant_opts(), row, col)
    P.assert_exact(row, oracle.quantize(synth.bits(x)), "cfg2 X row, full tensor")
    P.assert_exact(col, oracle.quantize(synth.bits(x), colwise=True), "cfg2 X col, full tensor")
    mask = synth.DEFAULT_RHT_SIGN_MASK
    for rounding in (B.ROUND_NEAREST_EVEN, B.ROUND_STOCHASTIC):
        B.nvfp4_quantize(xd, B.quant_opts(rounding=rounding, rht_colwise=True, rht_sign_mask=mask, seed=7, sr_offset=3),
                         row, col)
        check_copy_slabs(x, row, colwise=False, rounding=rounding, seed=7, sr_offset=3, what="cfg2 row")
        check_copy_slabs(x, col, colwise=True, rht=True, mask=mask, rounding=rounding, seed=7, sr_offset=3,
                         what="cfg2 col rotated")
    # only one copy requested
    B.nvfp4_quantize(xd, B.quant_opts(rounding=B.ROUND_STOCHASTIC, seed=7, sr_offset=3), None, col)
    check_copy_slabs(x, col, colwise=True, rounding=oracle.SR, seed=7, sr_offset=3, what="cfg2 col only")


def test_config4_squared_relu_input_and_long_contraction():
    """cfg 4 (FFN down-projection): half of X is exactly zero and the tail is heavy; K = 20480."""
    p = synth.config4(M=2048)  # a quarter of the tokens keeps the host-side generation short; K and N are full size
    M, N, K = p.M, p.N, p.K
    X, W = p.X.cuda(), p.W.cuda()
    X_row, X_col = B.alloc_tensor(M, K), B.alloc_tensor(K, M)
    W_row = B.alloc_tensor(N, K)
    B.nvfp4_quantize(X, B.quant_opts(rht_colwise=True, rht_sign_mask=p.rht_sign_mask), X_row, X_col)
    B.nvfp4_quantize(W, B.quant_opts(block_rows=16), W_row, None)
    check_copy_slabs(p.X, X_row, colwise=False, what="cfg4 X row")
    check_copy_slabs(p.X, X_col, colwise=True, rht=True, mask=p.rht_sign_mask, what="cfg4 X col")
    assert float((X_row.scales == 0).float().mean()) > 0  # all-zero blocks exist and are encoded as scale 0
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    B.nvfp4_gemm(X_row, W_row, Y)
    B.nvfp4_device_status()
    check_gemm_samples(Y, Operand(X_row, p.X, colwise=False), Operand(W_row, p.W, colwise=False, block_rows=16), True,
                       "cfg4 Fprop", 4)


def test_config5_qkv_projection_shapes():
    """cfg 5: the QKV projection 5120 -> 7168 at 16384 tokens (N = 7168 is not a power-of-two multiple)."""
    p = synth.config5_layer(0, M=4096)  # the GEMM tiling only depends on M through the number of row blocks
    M, N, K = p.M, p.N, p.K
    opts = B.quant_opts(rht_sign_mask=p.rht_sign_mask, seed=p.sr_seed, sr_offset=p.sr_offset)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    X, W, dY = p.X.cuda(), p.W.cuda(), p.dY.cuda()
    B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
    B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, dW, False, ws_b)
    B.nvfp4_device_status()
    X_row = B.alloc_tensor(M, K)
    B.nvfp4_quantize(X, B.quant_opts(), X_row, None)
    g_row, g_col = B.alloc_tensor(M, N), B.alloc_tensor(N, M)
    B.nvfp4_quantize(dY, B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=p.rht_sign_mask,
                                      seed=p.sr_seed, sr_offset=p.sr_offset), g_row, g_col)
    mask = p.rht_sign_mask
    sr = dict(rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset)
    check_gemm_samples(Y, Operand(X_row, p.X, colwise=False), Operand(W_row, p.W, colwise=False, block_rows=16), True,
                       "cfg5 qkv Fprop", 5)
    check_gemm_samples(dX, Operand(g_row, p.dY, colwise=False, **sr), Operand(W_col, p.W, colwise=True, block_rows=16),
                       True, "cfg5 qkv Dgrad", 6)
    check_gemm_samples(dW, Operand(g_col, p.dY, colwise=True, rht=True, mask=mask, **sr),
                       Operand(X_col, p.X, colwise=True, rht=True, mask=mask), False, "cfg5 qkv Wgrad", 7)


def test_config3_full_size_variants_bf16_layer_transform_sizes_error_metric():
    """The recipe's variants at the benchmark's size: the layer kept in BF16 (Section 4.1) on sampled rows x columns,
    dY quantized with the 4 x 4 and 128 x 128 transforms (Appendix E.4.2) on sampled slabs, and the error metric
    (Appendix E.2) of the full dY copy against sums the oracle forms from sampled slabs scaled to the tensor."""
    p = synth.config3()
    M, N, K = p.M, p.N, p.K
    X, W, dY = p.X.cuda(), p.W.cuda(), p.dY.cuda()
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros((N, K), dtype=torch.float32, device="cuda")
    B.nvfp4_linear_bf16_fwd(X, W, Y)
    B.nvfp4_linear_bf16_bwd(dY, X, W, K, dX, dW)
    B.nvfp4_device_status()
    rng = np.random.default_rng(5)
    f64 = lambda t: t.float().numpy().astype(np.float64)

    def sample(D, A, Bm, bf16, what):  # D = A Bm^T with A [rows x k], Bm [cols x k] given as CPU bf16 tensors
        rows = np.sort(rng.choice(A.shape[0], 12, replace=False))
        cols = np.sort(rng.choice(Bm.shape[0], 384, replace=False))
        Dref, T = oracle.gemm_tn(f64(A[rows]), f64(Bm[cols]))
        got = D[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy()
        tol = 1e-4 * T + (2.0 ** -8 * np.abs(Dref) if bf16 else 0.0) + 1e-30
        assert np.all(np.abs(got - Dref) <= tol), what

    sample(Y, p.X, p.W, True, "BF16 Fprop")
    sample(dX, p.dY, p.W.t().contiguous(), True, "BF16 Dgrad")
    sample(dW, p.dY.t().contiguous(), p.X.t().contiguous(), False, "BF16 Wgrad")

    # transform sizes on dY (stochastic rounding, plain row copy + rotated transposed copy)
    big_mask = 0x5A5A_73E5_1234_ABCD_0F0F_3C3C_9999_73E5
    g_row, g_col = B.alloc_tensor(M, N), B.alloc_tensor(N, M)
    for d in (4, 128):
        m = big_mask & ((1 << d) - 1)
        B.nvfp4_quantize(dY, B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=m, rht_dim=d,
                                          seed=p.sr_seed, sr_offset=p.sr_offset), g_row, g_col)
        check_copy_slabs(p.dY, g_row, colwise=False, rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset,
                         what=f"dY row beside d={d}")
        check_copy_slabs(p.dY, g_col, colwise=True, rht=True, mask=m, rounding=oracle.SR, seed=p.sr_seed,
                         sr_offset=p.sr_offset, what=f"dY col d={d}", rht_dim=d)

    # error metric of the row-wise copy: the oracle's sums over three 128-row slabs against the kernel's over the
    # same slabs (views of the full-size tensors), and the full-tensor value for plausibility
    for r0 in (0, M // 2, M - 128):
        ref = oracle.quantize(synth.bits(p.dY[r0:r0 + 128]), rounding=oracle.SR, seed=p.sr_seed, sr_offset=p.sr_offset,
                              amax_override=float(g_row.glob[0]), sr_row0=r0, sr_cols=N)
        e_ref, n_ref = oracle.quant_error(f64(p.dY[r0:r0 + 128]), oracle.dequantize(ref))
        # scale atoms of a 128-row slab are contiguous: rows r0 .. r0 + 127 form the atom row r0 / 128
        slab = B.NVFP4Tensor(g_row.codes[r0:r0 + 128], g_row.scales.view(-1)[(r0 // 128) * (N // 64) * 512:].contiguous(),
                             g_row.glob, 128, N, B.SF_SWIZZLED)
        out = B.nvfp4_quant_error(dY[r0:r0 + 128], slab).cpu().numpy()
        assert abs(out[0] - e_ref) <= 1e-5 * e_ref and abs(out[1] - n_ref) <= 1e-5 * n_ref, (r0, out, e_ref, n_ref)
    full = B.nvfp4_quant_error(dY, g_row).cpu().numpy()
    assert abs(full[1] - float((p.dY.double() ** 2).sum())) <= 1e-6 * full[1]
    assert 2e-3 < full[0] / full[1] < 5e-2
