"""Pins for the oracle's two-level scaling, block quantizer, Hadamard transform and GEMM (CPU only)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2509_25149_b200 import synth

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
F32 = np.float32


def f32_bits(x):
    return int(np.array([x], dtype=np.float32).view(np.uint32)[0])


def to_bits(values, shape):
    t = torch.tensor(values, dtype=torch.float32).reshape(shape)
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), t), "fixture values must be exact in bf16"
    return synth.bits(b)


def unpack(codes):
    lo, hi = codes & 15, codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


# ------------------------------------------------------- global scale, Eq. 1 ----
def test_global_scale_closed_forms():
    e, d = oracle.global_scale(2688.0)
    assert f32_bits(e) == 0x3F800000 and f32_bits(d) == 0x3F800000
    e, d = oracle.global_scale(1.0)
    assert e == F32(2688.0) and f32_bits(e) == 0x45280000
    assert d == F32(1.0) / F32(2688.0) and f32_bits(d) == 0x39C30C31
    e, d = oracle.global_scale(500.0)
    assert e == F32(2688.0) / F32(500.0) and d == F32(1.0) / e
    assert f32_bits(e) == 0x40AC0831 and f32_bits(d) == 0x3E3E79E8
    # s_dec is 1/s_enc, which is not always amax/2688 in the last bit: the order is part of the contract
    rng = np.random.default_rng(0)
    differ = 0
    for a in rng.uniform(0.01, 1000, 2000).astype(np.float32):
        e, d = oracle.global_scale(float(a))
        assert e == F32(2688.0) / a and d == F32(1.0) / e
        differ += d != a / F32(2688.0)
    assert differ > 100
    assert oracle.global_scale(0.0) == (F32(1.0), F32(1.0))
    e, d = oracle.global_scale(1e-42)  # 2688/denormal overflows -> clamped
    assert e == np.finfo(np.float32).max and d > 0


def test_block_scale_identity_and_range():
    # s_enc,b * s_dec * fp32(S_b) ~= 1 (text after Eq. 3); the largest block gets the FP8 maximum
    rng = np.random.default_rng(1)
    for amax in rng.uniform(1e-3, 1e4, 200).astype(np.float32):
        s_enc, s_dec = oracle.global_scale(float(amax))
        assert oracle.block_scale_byte(float(amax), s_enc) == 0x7E
        for amax_b in (amax * rng.uniform(2.0 ** -8, 1.0, 20)).astype(np.float32):
            sb = oracle.block_scale_byte(float(amax_b), s_enc)
            assert 0 < sb <= 0x7E
            enc_b = oracle.block_encode_scale(sb, s_dec)
            prod = float(enc_b) * float(s_dec) * oracle.e4m3_decode(sb)
            assert abs(prod - 1.0) <= 3 * 2.0 ** -24
            if oracle.e4m3_decode(sb) >= 2.0 ** -6:  # normal E4M3 scale: overshoot <= 6*(1+2^-4)
                assert float(amax_b) * float(enc_b) <= 6 * (1 + 2.0 ** -4) * (1 + 1e-6)
    s_enc, s_dec = oracle.global_scale(1.0)
    assert oracle.block_scale_byte(1e-7, s_enc) == 0 and oracle.block_encode_scale(0, s_dec) == 0.0


# --------------------------------------------------------- worked examples ----
def _worked_blocks():
    with open(os.path.join(GOLD, "worked_blocks.txt")) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    for i in range(0, len(lines), 4):
        name = lines[i]
        vals = [float(t) for t in lines[i + 1].split()]
        scales = [int(t, 16) for t in lines[i + 2].split()]
        codes = [int(t, 16) for t in lines[i + 3].split()]
        yield name, vals, scales, codes


@pytest.mark.parametrize("name,vals,scales,codes", list(_worked_blocks()), ids=lambda v: v if isinstance(v, str) else None)
def test_hand_worked_blocks(name, vals, scales, codes):
    x = to_bits(vals, (1, len(vals)))
    q = oracle.quantize(x)
    assert q.scales.reshape(-1).tolist() == scales
    assert unpack(q.codes).reshape(-1).tolist() == codes
    assert q.amax == max(abs(v) for v in vals)
    if name == "A":
        assert q.codes.reshape(-1)[:8].tolist() == [0x6F, 0x45, 0x24, 0x02, 0x90, 0x76, 0x06, 0x28]
        assert f32_bits(q.s_dec) == 0x3F800000
    if name == "C":
        # Appendix B.4: the same block under a power-of-two (rounded-up) scale would put amax on 3;
        # the E4M3 scale 0.5 puts it on the FP4 maximum
        d = oracle.dequantize(q)
        assert d[0, 0] == 3.0 and oracle.e2m1_decode(codes[0]) == 6.0


# ----------------------------------------------------- structural invariants ----
def _random_bits(shape, seed, scale=1.0, outliers=0.0):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(shape, generator=g) * scale
    if outliers:
        m = torch.rand(shape, generator=g) < outliers
        x = torch.where(m, x * 50, x)
    return synth.bits(x.to(torch.bfloat16))


def test_amax_element_of_every_block_is_recovered_to_fp8_precision():
    # Section 2 / Fig. 1: the block amax lands on the FP4 maximum and is recovered by the block scale
    x = _random_bits((64, 256), 1, outliers=0.01)
    xf = synth.from_bits(x).to(torch.float64).numpy()
    q = oracle.quantize(x)
    d = oracle.dequantize(q)
    codes = unpack(q.codes)
    blocks = xf.reshape(64, 16, 16)
    idx = np.abs(blocks).argmax(axis=2)
    r, b = np.meshgrid(np.arange(64), np.arange(16), indexing="ij")
    amax_vals = blocks[r, b, idx]
    amax_codes = codes.reshape(64, 16, 16)[r, b, idx]
    amax_deq = d.reshape(64, 16, 16)[r, b, idx]
    normal = np.vectorize(oracle.e4m3_decode)(q.scales) >= 2.0 ** -6
    assert np.all((amax_codes & 7)[normal] == 7)
    assert np.all(np.abs(amax_deq - amax_vals)[normal] <= 2.0 ** -4 * np.abs(amax_vals)[normal] * (1 + 1e-6))
    # the block that holds the tensor amax carries byte 0x7E
    i = np.unravel_index(np.abs(xf).argmax(), xf.shape)
    assert q.scales[i[0], i[1] // 16] == 0x7E
    # per-element RNE error bound in scaled units
    sb = np.vectorize(oracle.e4m3_decode)(q.scales).repeat(16, axis=1) * float(q.s_dec)
    ok = sb > 0
    v = np.where(ok, xf / np.where(ok, sb, 1), 0)
    err = np.abs(np.clip(v, -6, 6) - np.where(ok, d / np.where(ok, sb, 1), 0))
    bound = np.where(np.abs(v) < 2, 0.25, np.where(np.abs(v) < 4, 0.5, 1.0))
    assert np.all(err <= bound * (1 + 1e-5) + 1e-6)


def test_dequantize_identity_on_grid_and_idempotence():
    # tensors built on the NVFP4 grid: amax = 2688 * 2^-j (s_enc = 2^j exactly), block scales from the
    # E4M3 set, elements = grid value * scale * s_dec -> quantize must return the construction
    rng = np.random.default_rng(2)
    for j in (0, 3, 9):
        s_dec = 2.0 ** -j
        R, nb = 16, 8
        sbytes = rng.integers(0x28, 0x58, size=(R, nb)).astype(np.uint8)  # 2^-2 .. 2^3: products stay in bf16
        sbytes &= 0xF8  # power-of-two scales so that value*scale is exact in bf16's 8 bits
        sbytes[0, 0] = 0x7E
        codes = rng.integers(0, 16, size=(R, nb * 16)).astype(np.uint8)
        codes[:, ::16] = 7  # each block holds its maximum (6) so the scale is reproduced
        mags = np.array([oracle.e2m1_decode(c) for c in range(16)])
        sval = np.vectorize(oracle.e4m3_decode)(sbytes).repeat(16, axis=1)
        x = mags[codes] * sval * s_dec
        xb = torch.from_numpy(x).to(torch.bfloat16)
        assert torch.equal(xb.to(torch.float64), torch.from_numpy(x))
        q = oracle.quantize(synth.bits(xb))
        assert q.amax == F32(2688.0 * s_dec) and q.s_dec == F32(s_dec)
        assert np.array_equal(q.scales, sbytes)
        got = unpack(q.codes)
        same = (got == codes) | ((got & 7) == 0) & ((codes & 7) == 0)
        assert np.all(same) and np.array_equal(got & 7, codes & 7)
        d = oracle.dequantize(q)
        assert np.array_equal(d, x)
        q2 = oracle.quantize(synth.bits(torch.from_numpy(d).to(torch.bfloat16)))
        assert np.array_equal(q2.codes, q.codes) and np.array_equal(q2.scales, q.scales)


def test_zero_tensor_and_zero_blocks():
    q = oracle.quantize(np.zeros((16, 32), dtype=np.uint16))
    assert q.amax == 0 and q.s_dec == 1 and not q.scales.any() and not q.codes.any()
    x = to_bits([1.0] + [0.0] * 15 + [2.0 ** -20] * 16, (1, 32))  # second block underflows the E4M3 range
    q = oracle.quantize(x)
    assert q.scales.tolist() == [[0x7E, 0]] and not q.codes[0, 8:].any()
    assert np.all(oracle.dequantize(q)[0, 16:] == 0)


def test_colwise_copy_is_the_quantized_transpose():
    x = _random_bits((48, 80), 4, outliers=0.02)
    xt = np.ascontiguousarray(x.T)
    a, b = oracle.quantize(x, colwise=True), oracle.quantize(xt)
    assert a.rows == 80 and a.cols == 48
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales) and np.array_equal(a.glob, b.glob)
    # leading dimension larger than the row length
    wide = _random_bits((48, 96), 4)
    sub = wide[:, :80]
    c, d = oracle.quantize(sub), oracle.quantize(np.ascontiguousarray(sub))
    assert np.array_equal(c.codes, d.codes) and np.array_equal(c.scales, d.scales)


# ------------------------------------------------------ 2D weights, Sec. 4.3 ----
def test_2d_blocks_give_one_representation_for_both_passes():
    w = _random_bits((64, 96), 6, scale=0.02)
    row = oracle.quantize(w, block_rows=16)
    col = oracle.quantize(w, block_rows=16, colwise=True)
    assert np.array_equal(oracle.dequantize(row), oracle.dequantize(col).T)
    assert np.array_equal(unpack(row.codes), unpack(col.codes).T)
    assert np.array_equal(row.glob, col.glob)
    # one byte per 16x16 tile, replicated to its 16 rows
    t = row.scales.reshape(4, 16, 6)
    assert np.all(t == t[:, :1, :])
    # tile scale = scale of the tile's amax
    wf = synth.from_bits(w).to(torch.float32).numpy()
    s_enc, _ = oracle.global_scale(float(np.abs(wf).max()))
    tile_amax = np.abs(wf).reshape(4, 16, 6, 16).max(axis=(1, 3))
    want = np.vectorize(lambda a: oracle.block_scale_byte(float(a), s_enc))(tile_amax)
    assert np.array_equal(t[:, 0, :], want)
    # with 1x16 blocks along each pass's own contraction dimension the two representations differ
    r1, c1 = oracle.quantize(w), oracle.quantize(w, colwise=True)
    assert not np.array_equal(oracle.dequantize(r1), oracle.dequantize(c1).T)


# ------------------------------------------------------------ RHT, App. C ----
def _H():
    return np.array([[oracle.hadamard16_entry(j, k) for k in range(16)] for j in range(16)], dtype=np.float64)


def test_hadamard_matrix_properties():
    H = _H()
    assert np.array_equal(H @ H.T, 16 * np.eye(16))
    assert np.array_equal(H, H.T) and set(np.unique(H)) == {-1.0, 1.0}
    H2 = np.array([[1, 1], [1, -1]], dtype=np.float64)
    assert np.array_equal(H, np.kron(H2, np.kron(H2, np.kron(H2, H2))))
    # normalised recursion H_d = (1/sqrt 2) H_2 (x) H_{d/2}: four levels give the factor 1/4
    Hn = np.array([[1.0]])
    for _ in range(4):
        Hn = np.kron(H2, Hn) / np.sqrt(2)
    assert np.allclose(Hn, H / 4, atol=1e-15) and np.allclose(Hn @ Hn.T, np.eye(16), atol=1e-15)


def test_rht16_special_inputs():
    mask = 0x73E5
    s = np.array([-1.0 if (mask >> j) & 1 else 1.0 for j in range(16)])
    H = _H()
    for j in range(16):  # one-hot a*e_j -> s_j * a/4 * row j of H
        x = np.zeros(16, dtype=np.float32)
        x[j] = 3.0
        assert np.array_equal(oracle.rht16(x, mask), (0.75 * s[j] * H[j]).astype(np.float32))
    c = np.full(16, 2.5, dtype=np.float32)  # constant chunk, no signs -> (4c, 0, ..., 0)
    assert np.array_equal(oracle.rht16(c, 0), np.array([10.0] + [0.0] * 15, dtype=np.float32))
    rng = np.random.default_rng(8)
    x = rng.standard_normal(16).astype(np.float32)
    y = oracle.rht16(x, mask).astype(np.float64)
    assert np.allclose(y, (x * s) @ H / 4, rtol=0, atol=1e-6)
    assert abs(np.linalg.norm(y) - np.linalg.norm(x)) <= 1e-6  # Parseval
    back = (y @ H.T / 4) * s  # involution: (x S H)(H^T S) = x
    assert np.allclose(back, x, atol=1e-6)
    # the default sign mask is word 0 of Philox(key 0, counter (0,0,0,1)), low 16 bits
    assert int(oracle.philox4x32_10([0, 0, 0, 1], [0, 0])[0]) & 0xFFFF == synth.DEFAULT_RHT_SIGN_MASK


def test_rht_cancels_in_the_dot_product_before_quantization():
    # Eq. 6: (A H)(B H)^T = A B^T when both operands are rotated along the contraction dim
    a = _random_bits((32, 64), 9)
    b = _random_bits((48, 64), 10)
    mask = 0x73E5
    ya = oracle.quantize(a, rht=True, sign_mask=mask, return_y=True).y.astype(np.float64)
    yb = oracle.quantize(b, rht=True, sign_mask=mask, return_y=True).y.astype(np.float64)
    af = synth.from_bits(a).to(torch.float64).numpy()
    bf = synth.from_bits(b).to(torch.float64).numpy()
    assert np.allclose(ya @ yb.T, af @ bf.T, rtol=0, atol=1e-4)
    # a mismatched sign vector does not cancel
    yc = oracle.quantize(b, rht=True, sign_mask=mask ^ 1, return_y=True).y.astype(np.float64)
    assert not np.allclose(ya @ yc.T, af @ bf.T, rtol=0, atol=1e-2)


def test_rht_scales_live_in_the_rotated_space():
    # a constant chunk has rotated amax 4x the raw amax; the global scale must follow it
    x = to_bits([1.0] * 16 + [0.5] * 16, (2, 16))
    q = oracle.quantize(x, rht=True, sign_mask=0)
    assert q.amax == 4.0
    d = oracle.dequantize(q)
    # s_dec = 1/672 is not a power of two, so the decode is exact only to the "~= 1" of Appendix B.2
    assert abs(d[0, 0] - 4.0) <= 4 * 3 * 2.0 ** -24 and abs(d[1, 0] - 2.0) <= 2 * 3 * 2.0 ** -24
    assert not d[:, 1:].any() and unpack(q.codes)[:, 0].tolist() == [7, 7]
    assert q.scales.tolist() == [[0x7E], [0x76]]  # 448 and 224: the second block's rotated amax is half
    # column-wise copy: chunks run along the source rows
    xc = to_bits([1.0] * 16 * 16, (16, 16))
    qc = oracle.quantize(xc, colwise=True, rht=True, sign_mask=0)
    assert np.all(unpack(qc.codes)[:, 0] == 7) and not oracle.dequantize(qc)[:, 1:].any()
    # amax override is honoured (used by the GPU comparison protocol)
    q2 = oracle.quantize(x, rht=True, sign_mask=0, amax_override=8.0)
    assert q2.amax == 8.0 and q2.s_dec == oracle.global_scale(8.0)[1]


# ------------------------------------------------------------- SR, Sec. 4.4 ----
def test_sr_quantize_uses_source_position_draws_and_is_unbiased():
    x = _random_bits((32, 48), 12, scale=1e-3)
    rne = oracle.quantize(x)
    for colwise in (False, True):
        q = oracle.quantize(x, colwise=colwise, rounding=oracle.SR, seed=5, sr_offset=2, return_y=True)
        ref = oracle.quantize(x, colwise=colwise)
        assert np.array_equal(q.scales, ref.scales) and np.array_equal(q.glob, ref.glob)
        codes = unpack(q.codes)
        for (r, c) in [(0, 0), (3, 17), (31, 47), (16, 16), (5, 40)]:
            rr, cc = (c, r) if colwise else (r, c)  # position in the copy
            sb = oracle.block_encode_scale(int(q.scales[rr, cc // 16]), q.s_dec)
            v = F32(q.y[rr, cc]) * sb
            u = oracle.sr_draw(5, 2, r * 48 + c)  # keyed by the SOURCE row-major index
            assert codes[rr, cc] == oracle.e2m1_encode_sr(float(v), u)
    # row-wise and column-wise copies share the draw of a source element: same up/down decisions
    # wherever both copies happen to use the same block scale cannot be assumed, so only check means
    S = 1024
    acc = np.zeros((32, 48))
    for seed in range(S):
        acc += oracle.dequantize(oracle.quantize(x, rounding=oracle.SR, seed=seed))
    xf = synth.from_bits(x).to(torch.float64).numpy()
    sb = np.vectorize(oracle.e4m3_decode)(rne.scales).repeat(16, axis=1) * float(rne.s_dec)
    step = 2.0 * sb  # coarsest E2M1 step in real units
    # a block amax may overshoot 6 by up to 1/16 (its E4M3 scale rounded down) and then saturates: that
    # part of the error is deterministic, not rounding bias
    sat = np.maximum(np.abs(xf) - 6.0 * sb, 0.0)
    assert np.all(np.abs(acc / S - xf) <= sat + step * (1 / 512 + 2.5 / np.sqrt(S)) + 1e-12)
    # while RNE on such data has a systematic error the mean of SR does not share
    assert np.abs(acc / S - xf).mean() < 0.25 * np.abs(oracle.dequantize(rne) - xf).mean()


# ------------------------------------------------------------------- GEMM ----
def test_gemm_tn_against_numpy_and_exact_cases():
    rng = np.random.default_rng(13)
    A, B = rng.standard_normal((24, 80)), rng.standard_normal((40, 80))
    D, T = oracle.gemm_tn(A, B)
    assert np.allclose(D, A @ B.T, rtol=1e-13, atol=1e-13) and np.allclose(T, np.abs(A) @ np.abs(B).T, rtol=1e-13)
    # all ones -> every output equals K
    q = oracle.Quantized(np.full((32, 32), 0x22, np.uint8), np.full((32, 4), 0x38, np.uint8),
                         np.array([1.0, 1.0], np.float32), 32, 64)  # code 2 = 1.0, scale byte 0x38 = 1.0
    assert np.array_equal(oracle.gemm_blockscaled(q, q), np.full((32, 32), 64.0))
    assert np.array_equal(oracle.gemm_tn(oracle.dequantize(q), oracle.dequantize(q), want_T=False), np.full((32, 32), 64.0))


def test_eq5_blockwise_form_equals_product_of_decoded_operands():
    a = oracle.quantize(_random_bits((32, 128), 14, outliers=0.02))
    b = oracle.quantize(_random_bits((48, 128), 15, scale=0.02), block_rows=16)
    D, T = oracle.gemm_tn(oracle.dequantize(a), oracle.dequantize(b))
    D5 = oracle.gemm_blockscaled(a, b)
    assert np.all(np.abs(D - D5) <= 1e-13 * T)
    # linearity in one block scale: doubling it adds exactly that block's contribution
    b2 = oracle.Quantized(b.codes.copy(), b.scales.copy(), b.glob.copy(), b.rows, b.cols)
    old = int(b2.scales[5, 3])
    assert old >= 0x10
    b2.scales[5, 3] = old - 8  # previous binade of E4M3 = exactly half
    assert oracle.e4m3_decode(old - 8) == 0.5 * oracle.e4m3_decode(old)
    D2 = oracle.gemm_blockscaled(a, b2)
    da, db = oracle.dequantize(a), oracle.dequantize(b)
    contrib = -0.5 * (da[:, 48:64] @ db[5, 48:64])
    assert np.allclose(D2[:, 5] - D5[:, 5], contrib, rtol=0, atol=1e-12 * np.abs(T[:, 5]).max())
    assert np.array_equal(np.delete(D2, 5, axis=1), np.delete(D5, 5, axis=1))


def test_wgrad_rht_pipeline_stays_close_to_the_unquantized_product():
    # sanity of the whole Wgrad operand path (column-wise, RHT, SR on the gradient): the quantized
    # product approximates dY^T X; the rotation must cancel (a transposed or unrotated operand would not)
    p = synth.config1()
    X, dY = synth.bits(p.X)[:128, :64], synth.bits(p.dY)[:128, :48]
    xq = oracle.quantize(X, colwise=True, rht=True, sign_mask=p.rht_sign_mask)
    gq = oracle.quantize(dY, colwise=True, rht=True, sign_mask=p.rht_sign_mask, rounding=oracle.SR)
    dW, _ = oracle.gemm_tn(oracle.dequantize(gq), oracle.dequantize(xq))
    exact = p.dY[:128, :48].to(torch.float64).numpy().T @ p.X[:128, :64].to(torch.float64).numpy()
    rel = np.linalg.norm(dW - exact) / np.linalg.norm(exact)
    assert rel < 0.2
    bad = oracle.quantize(X, colwise=True, rht=False)
    dWbad, _ = oracle.gemm_tn(oracle.dequantize(gq), oracle.dequantize(bad))
    assert np.linalg.norm(dWbad - exact) / np.linalg.norm(exact) > 0.7


def test_row_slab_with_given_amax_equals_the_rows_of_the_full_tensor():
    # used by the full-size GPU tests: a slab of rows, quantized with the full tensor's amax and the slab's
    # position for the stochastic-rounding index, reproduces the corresponding part of either copy
    x = _random_bits((64, 48), 21, scale=1e-3)
    for rounding in (oracle.RNE, oracle.SR):
        full_r = oracle.quantize(x, rounding=rounding, seed=3, sr_offset=7)
        full_c = oracle.quantize(x, colwise=True, rounding=rounding, seed=3, sr_offset=7)
        slab = x[16:48]
        r = oracle.quantize(slab, rounding=rounding, seed=3, sr_offset=7, amax_override=float(full_r.amax), sr_row0=16, sr_cols=48)
        c = oracle.quantize(slab, colwise=True, rounding=rounding, seed=3, sr_offset=7, amax_override=float(full_c.amax),
                            sr_row0=16, sr_cols=48)
        assert np.array_equal(r.codes, full_r.codes[16:48]) and np.array_equal(r.scales, full_r.scales[16:48])
        assert np.array_equal(c.codes, full_c.codes[:, 8:24]) and np.array_equal(c.scales, full_c.scales[:, 1:3])


def test_column_slab_with_given_amax_equals_the_rows_of_the_transposed_copy():
    # also used by the full-size GPU tests: 16 source columns (a strided view), quantized with the full tensor's
    # amax and the slab's column offset for the draw index, reproduce 16 rows of the transposed copy and the
    # corresponding columns of the row-wise copy
    x = _random_bits((64, 48), 22, scale=1e-3)
    for rounding in (oracle.RNE, oracle.SR):
        for rht in (False, True):
            full_c = oracle.quantize(x, colwise=True, rht=rht, sign_mask=0x73E5, rounding=rounding, seed=3, sr_offset=7)
            slab = x[:, 16:32]
            assert slab.strides[0] == 96
            c = oracle.quantize(slab, colwise=True, rht=rht, sign_mask=0x73E5, rounding=rounding, seed=3, sr_offset=7,
                                amax_override=float(full_c.amax), sr_cols=48, sr_col0=16)
            assert np.array_equal(c.codes, full_c.codes[16:32]) and np.array_equal(c.scales, full_c.scales[16:32])
        full_r = oracle.quantize(x, block_rows=16, rounding=rounding, seed=3, sr_offset=7)
        r = oracle.quantize(x[:, 16:32], block_rows=16, rounding=rounding, seed=3, sr_offset=7,
                            amax_override=float(full_r.amax), sr_cols=48, sr_col0=16)
        assert np.array_equal(r.codes, full_r.codes[:, 8:16]) and np.array_equal(r.scales, full_r.scales[:, 1:2])


def test_binary32_source_follows_the_same_procedure():
    """Appendix B names FP32 as well as BF16 as the precision converted from: a binary32 source differs only in how the
    element is read."""
    x = _random_bits((32, 64), 31, scale=1.0)
    xf = synth.from_bits(x).float().numpy()
    for kw in (dict(), dict(colwise=True), dict(block_rows=16), dict(rounding=oracle.SR, seed=5),
               dict(colwise=True, rht=True, sign_mask=0x73E5)):
        a, b = oracle.quantize(x, **kw), oracle.quantize(xf, **kw)  # values exact in bf16: identical results
        assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
        assert a.glob.view(np.uint32).tolist() == b.glob.view(np.uint32).tolist()
    # a hand-worked block that bf16 could not hold: amax 2688 * (1 + 2^-20) -> s_enc = fl(2688 / amax) < 1
    blk = np.zeros((1, 16), dtype=np.float32)
    blk[0, :4] = [2688.0 * (1 + 2.0 ** -20), 1344.0, -448.0 * (1 + 2.0 ** -12), 3.0000002]
    q = oracle.quantize(blk)
    assert float(q.amax) == float(np.float32(2688.0 * (1 + 2.0 ** -20)))
    s_enc = np.float32(2688.0) / q.amax
    assert s_enc < 1 and float(q.s_dec) == float(np.float32(1.0) / s_enc)
    assert q.scales[0, 0] == 0x7E  # the block holding the tensor amax gets 448
    codes = [(q.codes[0, i // 2] >> (4 * (i & 1))) & 15 for i in range(4)]
    # v = x * fl(1 / (448 * s_dec)): 6 (amax), 3 (half of it), -1 - a little (rounds to -1), ~0.0067 (rounds to 0)
    assert [oracle.e2m1_decode(c) for c in codes] == [6.0, 3.0, -1.0, 0.0]
    # low mantissa bits matter: the same block rounded to bf16 first gives a different tensor amax
    qb = oracle.quantize(synth.bits(torch.from_numpy(blk).to(torch.bfloat16)))
    assert float(qb.amax) != float(q.amax)
