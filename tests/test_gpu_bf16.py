"""Parity of the BF16 GEMM / linear layer (the layers the recipe keeps in higher precision, Section 4.1 and
Appendix D) with the oracle's binary64 products, through the C ABI.

Tolerance: the tensor cores add exact bf16 products in FP32; with T = sum |a||b| the accumulated rounding error of a
contraction of length K <= 16384 stays below (K / 16) * 2^-24 * T < 1e-4 * T (one rounding per K = 16 instruction);
a bf16 output adds half an ulp of the result, 2^-8 |D|."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def assert_close(D, Dref, T, bf16_out, what=""):
    tol = 1e-4 * T + (2.0 ** -8 * np.abs(Dref) if bf16_out else 0.0) + 1e-30
    err = np.abs(D.astype(np.float64) - Dref)
    worst = np.unravel_index(np.argmax(err / tol), err.shape)
    assert np.all(err <= tol), f"{what}: worst at {worst}: got {D[worst]}, want {Dref[worst]}, tol {tol[worst]}"


def run(a, b, M, N, a_layout, b_layout, fp32, accumulate=False, D0=None):
    D = torch.full((M, N), float("nan"), dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
    if D0 is not None:
        D.copy_(D0)
    B.nvfp4_gemm_bf16(a.cuda(), b.cuda(), D, a_layout, b_layout, accumulate)
    B.nvfp4_device_status()
    return D.float().cpu().numpy()


LAYOUTS = [(B.K_MAJOR, B.K_MAJOR), (B.K_MAJOR, B.MN_MAJOR), (B.MN_MAJOR, B.K_MAJOR), (B.MN_MAJOR, B.MN_MAJOR)]


@pytest.mark.parametrize("a_layout,b_layout", LAYOUTS)
def test_exact_small_integers_every_layout(a_layout, b_layout):
    # entries in {-2..2}: every partial sum is an integer below 2^24, exact in FP32 in any order
    rng = np.random.default_rng(1)
    M, N, K = 512, 256, 320
    A = rng.integers(-2, 3, size=(M, K)).astype(np.float64)
    Bm = rng.integers(-2, 3, size=(N, K)).astype(np.float64)
    a = torch.tensor(A.T.copy() if a_layout == B.MN_MAJOR else A, dtype=torch.bfloat16)
    b = torch.tensor(Bm.T.copy() if b_layout == B.MN_MAJOR else Bm, dtype=torch.bfloat16)
    D = run(a, b, M, N, a_layout, b_layout, True)
    Dref = oracle.gemm_tn(A, Bm, want_T=False)
    assert np.array_equal(D.astype(np.float64), Dref)


def test_each_operand_element_lands_in_its_place():
    # one-hot probes: A = rows of the identity pattern, B random -> D reproduces B's columns (and vice versa),
    # which pins row / column / k order of both operand layouts independently of any summation
    M, N, K = 256, 256, 256
    rng = np.random.default_rng(2)
    Bm = rng.integers(-8, 9, size=(N, K)).astype(np.float64)
    perm = rng.permutation(K)
    A = np.zeros((M, K))
    A[np.arange(M), perm] = 1.0
    for a_layout, b_layout in LAYOUTS:
        a = torch.tensor(A.T.copy() if a_layout == B.MN_MAJOR else A, dtype=torch.bfloat16)
        b = torch.tensor(Bm.T.copy() if b_layout == B.MN_MAJOR else Bm, dtype=torch.bfloat16)
        D = run(a, b, M, N, a_layout, b_layout, True)
        assert np.array_equal(D.astype(np.float64), Bm[:, perm].T), (a_layout, b_layout)


@pytest.mark.parametrize("shape", [(256, 256, 64), (512, 768, 1088), (2560, 512, 4096)])
@pytest.mark.parametrize("fp32", [False, True])
def test_random_data_against_binary64(shape, fp32):
    M, N, K = shape
    x = synth.normal_with_outliers_bf16((M, K), 0.01, 20.0, 5, 6)
    w = synth.normal_bf16((N, K), 0.05, 7)
    Dref, T = oracle.gemm_tn(f64(x), f64(w))
    for a_layout, b_layout in LAYOUTS:
        a = x.t().contiguous() if a_layout == B.MN_MAJOR else x
        b = w.t().contiguous() if b_layout == B.MN_MAJOR else w
        assert_close(run(a, b, M, N, a_layout, b_layout, fp32), Dref, T, not fp32, f"{shape} {a_layout}{b_layout}")


def test_accumulate_and_leading_dimensions():
    M, N, K = 256, 512, 192
    x = synth.normal_bf16((M, K + 64), 1.0, 11)[:, :K]       # lda > K
    w = synth.normal_bf16((N, K + 8), 0.1, 12)[:, :K]
    Dref, T = oracle.gemm_tn(f64(x), f64(w))
    D0 = torch.randn((M, N + 32), generator=torch.Generator().manual_seed(3))
    buf = D0.cuda()
    B.nvfp4_gemm_bf16(x.cuda(), w.cuda(), buf[:, :N], accumulate=True)
    B.nvfp4_device_status()
    out = buf.cpu().numpy()
    assert_close(out[:, :N], Dref + D0[:, :N].numpy().astype(np.float64), T + np.abs(D0[:, :N].numpy()) * 1e-3, False)
    assert np.array_equal(out[:, N:], D0[:, N:].numpy()), "columns beyond N must stay untouched"
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_gemm_bf16(x.cuda(), w.cuda(), torch.empty((M, N), dtype=torch.bfloat16, device="cuda"), accumulate=True)
    with pytest.raises(B.NVFP4Error):
        B.nvfp4_gemm_bf16(x.cuda()[:124], w.cuda(), torch.empty((124, N), dtype=torch.bfloat16, device="cuda"))


@pytest.mark.parametrize("shape", [(8, 8, 8), (264, 136, 72), (1000, 520, 200), (136, 2056, 4104)])
def test_ragged_shapes_every_layout(shape):
    """M, N, K that are not multiples of the 256 x 256 x 64 tile: edges are zero-filled on load, clipped on store."""
    M, N, K = shape
    x = synth.normal_bf16((M, K), 1.0, 41)
    w = synth.normal_bf16((N, K), 0.1, 42)
    Dref, T = oracle.gemm_tn(f64(x), f64(w))
    for a_layout, b_layout in LAYOUTS:
        a = x.t().contiguous() if a_layout == B.MN_MAJOR else x
        b = w.t().contiguous() if b_layout == B.MN_MAJOR else w
        for fp32 in (False, True):
            # the output sits inside a larger buffer whose other elements must survive
            buf = torch.full((M + 8, N + 8), 7.0, dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
            B.nvfp4_gemm_bf16(a.cuda(), b.cuda(), buf[:M, :N], a_layout, b_layout)
            B.nvfp4_device_status()
            out = buf.float().cpu().numpy()
            assert_close(out[:M, :N], Dref, T, not fp32, f"{shape} {a_layout}{b_layout} fp32={fp32}")
            assert np.all(out[M:, :] == 7.0) and np.all(out[:, N:] == 7.0), "stores beyond M x N"


def test_linear_layer_fwd_bwd():
    M, N, K = 512, 768, 256
    x = synth.normal_with_outliers_bf16((M, K), 0.01, 20.0, 21, 22)
    w = synth.normal_bf16((N, K), 0.05, 23)
    dy = synth.normal_bf16((M, N), 0.02, 24)
    (Yref, TY) = oracle.linear_bf16_fwd(synth.bits(x), synth.bits(w))
    (dXref, TdX), (dWref, TdW) = oracle.linear_bf16_bwd(synth.bits(dy), synth.bits(x), synth.bits(w))
    X, W, G = x.cuda(), w.cuda(), dy.cuda()
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    B.nvfp4_linear_bf16_fwd(X, W, Y)
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.full((N, K), 0.5, dtype=torch.float32, device="cuda")
    B.nvfp4_linear_bf16_bwd(G, X, W, K, dX, dW, accumulate_dw=True)
    B.nvfp4_device_status()
    assert_close(Y.float().cpu().numpy(), Yref, TY, True, "Y")
    assert_close(dX.float().cpu().numpy(), dXref, TdX, True, "dX")
    assert_close(dW.cpu().numpy(), dWref + 0.5, TdW + 1e-3, False, "dW")
    # either output may be skipped
    dX2 = torch.empty_like(dX)
    B.nvfp4_linear_bf16_bwd(G, None, W, K, dX2, None)
    assert torch.equal(dX2, dX)


def test_many_tiles_per_pair_and_both_accumulators():
    # more tiles than CTA pairs, several rounds: exercises the alternation of the two accumulators and the ring
    M, N, K = 256 * 12, 256 * 14, 128
    rng = np.random.default_rng(9)
    A = rng.integers(-3, 4, size=(M, K)).astype(np.float64)
    Bm = rng.integers(-3, 4, size=(N, K)).astype(np.float64)
    D = run(torch.tensor(A, dtype=torch.bfloat16), torch.tensor(Bm, dtype=torch.bfloat16), M, N, B.K_MAJOR, B.K_MAJOR,
            True)
    assert np.array_equal(D.astype(np.float64), oracle.gemm_tn(A, Bm, want_T=False))  # integers: exact in FP32
