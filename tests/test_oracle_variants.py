"""Pins for the oracle's recipe variants: other Hadamard sizes (Appendix E.4.2), layers kept in BF16 (Section 4.1,
Appendix D) and the quantization-error metric (Appendix E.2).  Each is checked against something the mathematics
fixes: Kronecker structure, orthogonality, closed forms, bilinearity of the layer, hand-computed sums."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2509_25149_b200 import synth

H2 = np.array([[1.0, 1.0], [1.0, -1.0]])


def sylvester(d):
    H = np.array([[1.0]])
    while H.shape[0] < d:
        H = np.kron(H2, H)
    return H


def signs(mask, d):
    return np.array([-1.0 if (mask >> j) & 1 else 1.0 for j in range(d)])


@pytest.mark.parametrize("d", [2, 4, 8, 16, 32, 64, 128])
def test_rht_d_is_the_normalised_sylvester_matrix_with_input_signs(d):
    rng = np.random.default_rng(d)
    mask = int.from_bytes(rng.bytes(16), "little") & ((1 << d) - 1)
    x = rng.standard_normal(d).astype(np.float32)
    y = oracle.rht_d(x, d, mask)
    H = sylvester(d)
    assert np.array_equal(H @ H.T, d * np.eye(d)) and np.array_equal(H, H.T)
    ref = (signs(mask, d) * x.astype(np.float64)) @ H / math.sqrt(d)
    assert np.allclose(y, ref, rtol=0, atol=2e-7 * np.abs(x).sum())
    # orthogonal: norms are kept, and applying H / sqrt(d) again (then the signs) returns the input
    assert abs(np.linalg.norm(y.astype(np.float64)) - np.linalg.norm(x.astype(np.float64))) < 1e-5
    back = (y.astype(np.float64) @ H / math.sqrt(d)) * signs(mask, d)
    assert np.allclose(back, x, atol=1e-5)
    # one non-zero input picks one (signed) row of the matrix
    one = np.zeros(d, dtype=np.float32)
    one[d - 1] = 3.0
    assert np.allclose(oracle.rht_d(one, d, mask), 3.0 / math.sqrt(d) * signs(mask, d)[d - 1] * H[d - 1], rtol=1e-7)
    # a constant chunk collapses onto the first output
    const = oracle.rht_d(np.full(d, 2.0, dtype=np.float32), d, 0)
    assert np.isclose(const[0], 2.0 * math.sqrt(d), rtol=1e-7) and np.all(const[1:] == 0.0)


def test_rht_d_special_sizes():
    x = np.random.default_rng(1).standard_normal(16).astype(np.float32)
    for mask in (0, 0x73E5, 0xFFFF, 0x8001):
        assert np.array_equal(oracle.rht_d(x, 16, mask), oracle.rht16(x, mask))
    # d = 2 by hand: [1, 2] -> [3, -1] / sqrt 2; with the second input negated -> [-1, 3] / sqrt 2
    assert np.allclose(oracle.rht_d(np.float32([1, 2]), 2, 0), [3 / math.sqrt(2), -1 / math.sqrt(2)], rtol=1e-7)
    assert np.allclose(oracle.rht_d(np.float32([1, 2]), 2, 2), [-1 / math.sqrt(2), 3 / math.sqrt(2)], rtol=1e-7)
    # d = 4 on small integers is exact (normalisation 1/2)
    assert np.array_equal(oracle.rht_d(np.float32([1, 2, 3, 4]), 4, 0), np.float32([5, -1, -2, 0]))
    for d in (1, 3, 256):
        with pytest.raises(ValueError):
            oracle.rht_d(np.zeros(d, dtype=np.float32), d, 0)


@pytest.mark.parametrize("d", [2, 4, 128])
def test_transform_cancels_in_the_contraction(d):
    """Section 4.2 / Appendix C: both Wgrad operands are rotated along the contraction dimension with the same
    matrix, which is orthogonal, so the product is unchanged."""
    rng = np.random.default_rng(3)
    mask = int.from_bytes(rng.bytes(16), "little") & ((1 << d) - 1)
    A = rng.standard_normal((5, 2 * d)).astype(np.float32)
    B = rng.standard_normal((3, 2 * d)).astype(np.float32)
    rot = lambda M: np.stack([np.concatenate([oracle.rht_d(r[c:c + d], d, mask) for c in range(0, 2 * d, d)]) for r in M])
    assert np.allclose(rot(A).astype(np.float64) @ rot(B).astype(np.float64).T,
                       A.astype(np.float64) @ B.astype(np.float64).T, atol=2e-4)


@pytest.mark.parametrize("d,colwise", [(4, False), (4, True), (16, True)])
def test_quantize_with_an_exact_transform_equals_quantizing_the_rotated_tensor(d, colwise):
    """With small-integer inputs and d = 4 or 16 the rotated values are exact bf16 numbers, so quantizing with the
    transform must give the very bytes of quantizing the explicitly rotated tensor without it."""
    rng = np.random.default_rng(5)
    mask = 0x73E5 & ((1 << d) - 1)
    x = rng.integers(-3, 4, size=(32, 64)).astype(np.float64)
    xb = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)
    src = x.T if colwise else x  # the copy: blocks run along its columns
    H = sylvester(d) / math.sqrt(d)
    rot = np.concatenate([(signs(mask, d) * src[:, c:c + d]) @ H for c in range(0, src.shape[1], d)], axis=1)
    rb = torch.tensor(rot, dtype=torch.float32).to(torch.bfloat16)
    assert np.array_equal(rb.float().numpy().astype(np.float64), rot), "rotated values must be exact in bf16"
    a = oracle.quantize(synth.bits(xb), colwise=colwise, rht=True, sign_mask=mask, rht_dim=d, return_y=True)
    b = oracle.quantize(synth.bits(rb))
    assert np.array_equal(a.y.astype(np.float64), rot)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales) and np.array_equal(a.glob, b.glob)


def test_quantize_transform_sizes_differ_and_need_whole_chunks():
    x = synth.normal_with_outliers_bf16((128, 256), 0.01, 30.0, 21, 22)
    ys = {d: oracle.quantize(synth.bits(x), rht=True, sign_mask=0x5A5A_73E5_1234_ABCD_0F0F_3C3C_9999_73E5 & ((1 << d) - 1),
                             rht_dim=d, return_y=True) for d in (2, 4, 8, 16, 128)}
    xf = x.float().numpy().astype(np.float64)
    for d, q in ys.items():
        # every size keeps the row norms (orthogonal per chunk)
        assert np.allclose(np.linalg.norm(q.y.astype(np.float64), axis=1), np.linalg.norm(xf, axis=1), rtol=1e-5)
    # a larger transform spreads an outlier over more elements: the amax of the rotated tensor shrinks with d
    amax = [float(ys[d].glob[0]) for d in (2, 4, 16, 128)]
    assert amax[0] > amax[1] > amax[2] > amax[3]
    with pytest.raises(ValueError):
        oracle.quantize(synth.bits(synth.normal_bf16((16, 64), 1.0, 1)), rht=True, rht_dim=128)
    with pytest.raises(ValueError):
        oracle.quantize(synth.bits(x), rht=True, rht_dim=4, block_rows=16)


# ------------------------------------------------------------ BF16 layer ----
def test_bf16_layer_definitions_and_gradient_identities():
    M, N, K = 24, 40, 56
    x = synth.normal_bf16((M, K), 1.0, 31)
    w = synth.normal_bf16((N, K), 0.05, 32)
    dy = synth.normal_bf16((M, N), 0.1, 33)
    X, W, G = (t.float().numpy().astype(np.float64) for t in (x, w, dy))
    Y, T = oracle.linear_bf16_fwd(synth.bits(x), synth.bits(w))
    assert np.allclose(Y, X @ W.T, rtol=1e-13, atol=1e-13) and np.allclose(T, np.abs(X) @ np.abs(W).T, rtol=1e-13)
    (dX, TdX), (dW, TdW) = oracle.linear_bf16_bwd(synth.bits(dy), synth.bits(x), synth.bits(w))
    assert dX.shape == (M, K) and dW.shape == (N, K)
    # L = <dY, Y> is bilinear in (X, W): its change along any direction is exactly <dX, E> resp. <dW, F>
    rng = np.random.default_rng(34)
    E, F = rng.standard_normal((M, K)), rng.standard_normal((N, K))
    L = lambda Xv, Wv: float(np.sum(G * (Xv @ Wv.T)))
    assert math.isclose(L(X + E, W) - L(X, W), float(np.sum(dX * E)), rel_tol=1e-9, abs_tol=1e-9)
    assert math.isclose(L(X, W + F) - L(X, W), float(np.sum(dW * F)), rel_tol=1e-9, abs_tol=1e-9)
    # element by hand
    assert math.isclose(dX[3, 5], sum(G[3, n] * W[n, 5] for n in range(N)), rel_tol=1e-12)
    assert math.isclose(dW[7, 2], sum(G[m, 7] * X[m, 2] for m in range(M)), rel_tol=1e-12)
    assert np.allclose(TdX, np.abs(G) @ np.abs(W), rtol=1e-13) and np.allclose(TdW, np.abs(G).T @ np.abs(X), rtol=1e-13)


# ------------------------------------------------------ error metric ----
def test_quant_error_by_hand_and_on_the_grid():
    assert oracle.quant_error([1.0, 2.0, 3.0], [1.0, 2.5, 2.0]) == (1.25, 14.0)
    # values on the quantization grid decode to themselves up to the rounding of the tensor decode scale (1/448 is
    # not a binary32 number): no quantization error
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    rng = np.random.default_rng(41)
    v = rng.choice(grid, size=(16, 64)) * rng.choice([-1.0, 1.0], size=(16, 64))
    v[:, ::16] = 6.0
    xb = torch.tensor(v, dtype=torch.float32).to(torch.bfloat16)
    err, ref = oracle.quant_error(v, oracle.dequantize(oracle.quantize(synth.bits(xb))))
    assert err <= 1e-13 * ref and ref == float(np.sum(v * v))
    # random data: the relative error of 4-bit quantization with 16-element blocks sits near 1e-2, and stochastic
    # rounding, being unbiased but noisier, has the larger squared error
    x = synth.normal_bf16((64, 256), 1.0, 42)
    xf = x.float().numpy().astype(np.float64)
    e_rne, n = oracle.quant_error(xf, oracle.dequantize(oracle.quantize(synth.bits(x))))
    e_sr, _ = oracle.quant_error(xf, oracle.dequantize(oracle.quantize(synth.bits(x), rounding=oracle.SR, seed=1)))
    assert 2e-3 < e_rne / n < 3e-2 and e_rne < e_sr < 4 * e_rne


# ------------------------------------------- row-granular global scale ----
def test_rowscale_reduces_to_the_tensor_scale_and_decouples_rows():
    """Appendix B.1's closing remark: a global scale per row.  Pins: rows sharing one amax give the tensor-scaled
    result bit for bit; a row's bytes do not depend on the other rows; an outlier row no longer costs the small
    rows their resolution; on-grid rows decode exactly; SR draws are those of the whole-tensor positions."""
    x = synth.normal_bf16((32, 256), 1.0, 91)
    xb = synth.bits(x).copy()
    # (a) give every row the same maximum: per-row scaling must equal per-tensor scaling
    top = np.uint16(0x4120)  # 10.0 in bf16, above every N(0,1) sample
    xb[:, 7] = top
    a = oracle.quantize_rowscale(xb)
    b = oracle.quantize(xb)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
    assert np.all(a.glob == b.glob[None, :])
    # (b) rows are independent: changing row 3 leaves all other rows' bytes alone
    xb2 = xb.copy()
    xb2[3, 100] = np.uint16(0x447A)  # 1000.0
    c = oracle.quantize_rowscale(xb2)
    keep = np.arange(32) != 3
    assert np.array_equal(c.codes[keep], a.codes[keep]) and np.array_equal(c.glob[keep], a.glob[keep])
    assert c.glob[3, 0] == 1000.0
    # (c) with a per-tensor scale the same outlier flushes small blocks of OTHER rows to zero, with row scales not
    small = synth.normal_bf16((8, 64), 1e-4, 92)
    sb = synth.bits(small).copy()
    sb[0, 0] = np.uint16(0x4F00)  # 2^31 in row 0
    xs = synth.from_bits(sb).to(torch.float64).numpy()
    e_tensor = np.abs(oracle.dequantize(oracle.quantize(sb)) - xs)[1:].max()
    e_rows = np.abs(oracle.dequantize_rowscale(oracle.quantize_rowscale(sb)) - xs)[1:].max()
    assert e_rows < 0.2 * np.abs(xs[1:]).max() and e_tensor == np.abs(xs[1:]).max(), (e_rows, e_tensor)  # flushed to zero
    # (d) stochastic rounding: row r of the row-scaled copy is the 1-row tensor quantized with the draws of the
    # positions (r, c) of the whole source
    q = oracle.quantize_rowscale(xb, rounding=oracle.SR, seed=5, sr_offset=2)
    one = oracle.quantize(xb[9:10], rounding=oracle.SR, seed=5, sr_offset=2, sr_row0=9, sr_cols=256)
    assert np.array_equal(q.codes[9], one.codes[0])
    v = oracle.dequantize_rowscale(q)
    assert np.all(np.abs(v - synth.from_bits(xb).to(torch.float64).numpy()) <= 2.0 * 10.0 / 6 * 1.07)
