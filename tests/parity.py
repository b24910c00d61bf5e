"""Comparison protocol between the CUDA path (through the C ABI) and the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

E4M3_VALUES = np.array([oracle.e4m3_decode(i) for i in range(0x7F)], dtype=np.float64)
E4M3_MIDPOINTS = (E4M3_VALUES[1:] + E4M3_VALUES[:-1]) / 2
E2M1_GRID = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
E2M1_MIDPOINTS = (E2M1_GRID[1:] + E2M1_GRID[:-1]) / 2


def unpack(codes: np.ndarray) -> np.ndarray:
    return np.stack([codes & 15, codes >> 4], axis=-1).reshape(codes.shape[0], -1)


def download(t: B.NVFP4Tensor):
    """GPU copy -> (codes [R][C/2], scales linear [R][C/16], glob[2]) as numpy."""
    torch.cuda.synchronize()
    codes = t.codes.cpu().numpy()
    sc = t.scales.cpu().numpy()
    if t.sf_layout == B.SF_SWIZZLED:
        sc = oracle.sf_unswizzle(sc, t.rows, t.cols // 16)
    else:
        sc = sc.reshape(t.rows, t.cols // 16)
    return codes, sc, t.glob.cpu().numpy()


def upload(q: oracle.Quantized, device="cuda") -> B.NVFP4Tensor:
    """Oracle copy -> device tensors in the swizzled scale layout the GEMM reads."""
    return B.NVFP4Tensor(torch.from_numpy(np.ascontiguousarray(q.codes)).to(device),
                         torch.from_numpy(oracle.sf_swizzle(q.scales)).to(device),
                         torch.from_numpy(np.ascontiguousarray(q.glob)).to(device), q.rows, q.cols, B.SF_SWIZZLED)


def upload_linear(q: oracle.Quantized, device="cuda") -> B.NVFP4Tensor:
    """Oracle copy -> device tensors with the scales in the plain [rows][blocks] layout."""
    return B.NVFP4Tensor(torch.from_numpy(np.ascontiguousarray(q.codes)).to(device),
                         torch.from_numpy(np.ascontiguousarray(q.scales)).to(device),
                         torch.from_numpy(np.ascontiguousarray(q.glob)).to(device), q.rows, q.cols, B.SF_LINEAR)


def gpu_quantize(x: torch.Tensor, *, rowwise=True, colwise=False, sf_layout=B.SF_SWIZZLED, **opt):
    """x: CPU bf16 tensor.  Returns (row copy or None, col copy or None) as device NVFP4Tensors."""
    xd = x.cuda()
    R, C = x.shape
    row = B.alloc_tensor(R, C, sf_layout) if rowwise else None
    col = B.alloc_tensor(C, R, sf_layout) if colwise else None
    B.nvfp4_quantize(xd, B.quant_opts(**opt), row, col)
    torch.cuda.synchronize()
    return row, col


def assert_exact(gpu: B.NVFP4Tensor, ref: oracle.Quantized, what=""):
    codes, scales, glob = download(gpu)
    assert glob.view(np.uint32).tolist() == ref.glob.view(np.uint32).tolist(), f"{what}: global {glob} vs {ref.glob}"
    bad = np.argwhere(scales != ref.scales)
    assert bad.size == 0, f"{what}: {len(bad)} scale bytes differ, first at {bad[0]}: " \
                          f"{scales[tuple(bad[0])]:#x} vs {ref.scales[tuple(bad[0])]:#x}"
    bad = np.argwhere(codes != ref.codes)
    assert bad.size == 0, f"{what}: {len(bad)} code bytes differ, first at {bad[0]}: " \
                          f"{codes[tuple(bad[0])]:#x} vs {ref.codes[tuple(bad[0])]:#x}"


def canon_zero(nibbles: np.ndarray) -> np.ndarray:
    """E2M1 has two zeros (codes 0 and 8).  Which one a transformed element gets depends on the order in which
    signed zeros are added, which no passage fixes; they decode to the same value, so compare them as equal."""
    out = nibbles.copy()
    out[out == 8] = 0
    return out


def assert_exact_up_to_zero_sign(gpu: B.NVFP4Tensor, ref: oracle.Quantized, what=""):
    """Bit-exact scales and tensor words; codes equal except that -0 and +0 are the same code."""
    codes, scales, glob = download(gpu)
    assert glob.view(np.uint32).tolist() == ref.glob.view(np.uint32).tolist(), f"{what}: global {glob} vs {ref.glob}"
    assert np.array_equal(scales, ref.scales), f"{what}: scale bytes"
    bad = np.argwhere(canon_zero(unpack(codes)) != canon_zero(unpack(ref.codes)))
    assert bad.size == 0, f"{what}: {len(bad)} codes differ, first at {bad[0]}"


def assert_rht_close(x_bits: np.ndarray, gpu: B.NVFP4Tensor, y_gpu, *, colwise, sign_mask, rounding,
                     seed=0, sr_offset=0, what="", rht_dim=16):
    """Tolerance protocol for transformed copies (the transform is computed in a different order on the GPU):
    values within 1e-5 of the scale of their dot product; amax within 1e-5; then, with the oracle re-run on the
    GPU's amax, scale bytes equal except where the pre-rounding scale is within 1e-5 of an E4M3 midpoint, and
    codes equal except where the pre-rounding value is within 1e-5 of a rounding threshold (an excused code must
    still be an adjacent grid point).  Excused items must stay below 1e-3 of all elements.
    y_gpu may be None (no device-side dump of the transformed values for that transform size): step (1) is skipped."""
    codes, scales, glob = download(gpu)
    d = rht_dim
    ref0 = oracle.quantize(x_bits, colwise=colwise, rht=True, sign_mask=sign_mask, rounding=rounding, seed=seed,
                           sr_offset=sr_offset, return_y=True, rht_dim=d)
    # (1) transformed values
    if y_gpu is not None:
        xs = synth.from_bits(x_bits).to(torch.float64).numpy()
        src = xs.T if colwise else xs
        l1 = np.abs(src).reshape(src.shape[0], -1, d).sum(axis=2).repeat(d, axis=1) / np.sqrt(d)
        assert np.all(np.abs(y_gpu.astype(np.float64) - ref0.y) <= 1e-5 * l1 + 1e-30), f"{what}: transformed values"
    # (2) amax
    assert abs(float(glob[0]) - float(ref0.amax)) <= 1e-5 * float(ref0.amax), f"{what}: amax"
    ref = oracle.quantize(x_bits, colwise=colwise, rht=True, sign_mask=sign_mask, rounding=rounding, seed=seed,
                          sr_offset=sr_offset, amax_override=float(glob[0]), return_y=True, rht_dim=d)
    assert glob.view(np.uint32).tolist() == ref.glob.view(np.uint32).tolist(), f"{what}: s_dec from the same amax"
    counts = compare_rotated(codes, scales, ref, float(glob[0]), rounding,
                             lambda r, c: oracle.sr_draw(seed, sr_offset, (c if colwise else r) * x_bits.shape[1] +
                                                         (r if colwise else c)), what)
    total = ref.rows * ref.cols
    assert counts["excused_codes"] + 16 * counts["excused_scales"] <= max(1e-3 * total, 16), f"{what}: too many excused items"
    counts["elements"] = total
    return counts


def compare_rotated(codes, scales, ref, amax, rounding, draw, what=""):
    """Steps (3) and (4) of the protocol for transformed copies, on a whole copy or on a slab of one.
    codes / scales: the GPU's bytes (scales in the linear layout); ref: the oracle's copy of the same elements made
    with the GPU's tensor amax and `return_y=True`; draw(r, c): the 8-bit draw of element (r, c) of the copy.
    Scale bytes must be equal except where the pre-rounding scale is within 1e-5 of an E4M3 midpoint (then adjacent);
    codes, in blocks whose scale agrees, equal except where the pre-rounding value is within 1e-5 of a rounding
    threshold (then an adjacent grid point).  Returns the number of excused codes and scale bytes."""
    s_enc, s_dec = oracle.global_scale(amax)
    R, C = ref.rows, ref.cols
    amax_b = np.abs(ref.y).reshape(R, C // 16, 16).max(axis=2)
    t_b = ((amax_b.astype(np.float32) / np.float32(6)) * np.float32(s_enc)).astype(np.float64)
    nearest_mid = E4M3_MIDPOINTS[np.clip(np.searchsorted(E4M3_MIDPOINTS, t_b), 0, len(E4M3_MIDPOINTS) - 1)]
    prev_mid = E4M3_MIDPOINTS[np.clip(np.searchsorted(E4M3_MIDPOINTS, t_b) - 1, 0, len(E4M3_MIDPOINTS) - 1)]
    near = np.minimum(np.abs(t_b - nearest_mid), np.abs(t_b - prev_mid)) <= 1e-5 * np.maximum(t_b, 1e-30)
    sdiff = scales != ref.scales
    assert not np.any(sdiff & ~near), f"{what}: {np.count_nonzero(sdiff & ~near)} unexcused scale bytes"
    assert np.all(np.abs(scales.astype(int) - ref.scales.astype(int))[sdiff] == 1), f"{what}: excused scale not adjacent"
    # codes in blocks whose scale agrees
    got, want = canon_zero(unpack(codes)), canon_zero(unpack(ref.codes))
    cdiff = (got != want) & ~np.repeat(sdiff, 16, axis=1)
    excused = 0
    for r, c in np.argwhere(cdiff):
        enc_b = oracle.block_encode_scale(int(ref.scales[r, c // 16]), s_dec)
        v = float(np.float32(ref.y[r, c]) * enc_b)
        a = min(abs(v), 6.0)
        if rounding == oracle.RNE:
            thr = E2M1_MIDPOINTS
            step = 0.5 if a < 2 else (1.0 if a < 4 else 2.0)
        else:
            u = draw(int(r), int(c))
            lo = E2M1_GRID[E2M1_GRID <= a].max()
            hi = E2M1_GRID[E2M1_GRID > a].min() if a < 6 else 6.0
            step = max(hi - lo, 0.5)
            thr = np.array([lo + (hi - lo) * (u + 0.5) / 256])
        assert np.min(np.abs(thr - a)) <= 1e-5 * max(a, step), f"{what}: code at {(r, c)} differs away from a threshold (v={v})"
        assert abs(int(got[r, c] & 7) - int(want[r, c] & 7)) <= 1, f"{what}: excused code not adjacent"
        excused += 1
    # blocks with an excused scale: decoded values still within one E2M1 step (in the block's own scale) of y
    if np.any(sdiff):
        glob = np.array([amax, s_dec], dtype=np.float32)
        deq = oracle.dequantize(oracle.Quantized(np.ascontiguousarray(codes), np.ascontiguousarray(scales), glob, R, C))
        sb = np.vectorize(oracle.e4m3_decode)(scales).repeat(16, axis=1) * float(s_dec)
        m = np.repeat(sdiff, 16, axis=1)
        assert np.all(np.abs(deq - ref.y)[m] <= 2.0 * sb[m] * (1 + 2.0 ** -3) + 1e-30), f"{what}: excused block decode"
    return {"excused_codes": excused, "excused_scales": int(np.count_nonzero(sdiff))}


def decode_rows(t: B.NVFP4Tensor, rows) -> np.ndarray:
    """FP64 decode, by the oracle, of sampled rows of a device copy: the very bytes the GEMM reads."""
    torch.cuda.synchronize()
    rows = np.asarray(rows, dtype=np.int64)
    codes = t.codes[torch.from_numpy(rows).to(t.codes.device)].cpu().numpy()
    sc = t.scales.cpu().numpy()
    sc = oracle.sf_unswizzle(sc, t.rows, t.cols // 16) if t.sf_layout == B.SF_SWIZZLED else sc.reshape(t.rows, t.cols // 16)
    q = oracle.Quantized(np.ascontiguousarray(codes), np.ascontiguousarray(sc[rows]), t.glob.cpu().numpy(), len(rows), t.cols)
    return oracle.dequantize(q)


def gemm_reference(a: oracle.Quantized, b: oracle.Quantized, rows=None, cols=None):
    """FP64 product of the decoded operands and its tolerance scale, optionally on a subset of rows / columns."""
    da, db = oracle.dequantize(a), oracle.dequantize(b)
    if rows is not None:
        da = da[rows]
    if cols is not None:
        db = db[cols]
    return oracle.gemm_tn(da, db)


def assert_gemm_close(D: np.ndarray, Dref: np.ndarray, T: np.ndarray, bf16_out: bool, what=""):
    tol = 1e-3 * T + (2.0 ** -8 * np.abs(Dref) if bf16_out else 0.0) + 1e-30
    err = np.abs(D.astype(np.float64) - Dref)
    worst = np.unravel_index(np.argmax(err / tol), err.shape)
    assert np.all(err <= tol), f"{what}: worst at {worst}: got {D[worst]}, want {Dref[worst]}, tol {tol[worst]}"
    return float((err / np.maximum(T, 1e-300)).max())


# ------------------------------------------------------------------ MXFP4 (comparison format) ----
def download_mx(t: B.NVFP4Tensor):
    """GPU MXFP4 copy -> (codes [R][C/2], UE8M0 scales linear [R][C/32]) as numpy."""
    torch.cuda.synchronize()
    codes = t.codes.cpu().numpy()
    sc = t.scales.cpu().numpy()
    sc = oracle.sf_unswizzle(sc, t.rows, t.cols // 32) if t.sf_layout == B.SF_SWIZZLED else sc.reshape(t.rows, t.cols // 32)
    g = t.glob.cpu().numpy()
    assert g.tolist() == [0.0, 1.0], "an MXFP4 copy has no tensor-level scale"
    return codes, sc


def gpu_quantize_mx(x: torch.Tensor, *, rowwise=True, colwise=False, sf_layout=B.SF_SWIZZLED, **opt):
    xd = x.cuda()
    R, C = x.shape
    row = B.alloc_tensor(R, C, sf_layout, format=B.FORMAT_MXFP4) if rowwise else None
    col = B.alloc_tensor(C, R, sf_layout, format=B.FORMAT_MXFP4) if colwise else None
    B.nvfp4_quantize(xd, B.quant_opts(**opt), row, col)
    torch.cuda.synchronize()
    return row, col


def assert_exact_mx(gpu: B.NVFP4Tensor, ref: oracle.QuantizedMX, what=""):
    codes, scales = download_mx(gpu)
    bad = np.argwhere(scales != ref.scales)
    assert bad.size == 0, f"{what}: {len(bad)} scale bytes differ, first at {bad[0]}: " \
                          f"{scales[tuple(bad[0])]} vs {ref.scales[tuple(bad[0])]}"
    bad = np.argwhere(codes != ref.codes)
    assert bad.size == 0, f"{what}: {len(bad)} code bytes differ, first at {bad[0]}: " \
                          f"{codes[tuple(bad[0])]:#x} vs {ref.codes[tuple(bad[0])]:#x}"


def assert_mx_rht_close(x_bits: np.ndarray, gpu: B.NVFP4Tensor, *, colwise, sign_mask, rounding, seed=0, sr_offset=0,
                        what=""):
    """Tolerance protocol for transformed MXFP4 copies (the GPU sums in FP32 and multiplies by fl(1/sqrt(32)), the
    oracle rounds the exact value once): scale bytes equal except where amax_b / 6 is within 1e-5 of a power of two
    (an excused byte is adjacent); codes, in blocks whose scale agrees, equal except where the scaled value is
    within 1e-5 of a rounding threshold (an excused code is an adjacent grid point).  Excused items must stay below
    1e-3 of all elements."""
    codes, scales = download_mx(gpu)
    ref = oracle.quantize_mx(x_bits, colwise=colwise, rht=True, sign_mask=sign_mask, rounding=rounding, seed=seed,
                             sr_offset=sr_offset, return_y=True)
    R, C = ref.rows, ref.cols
    amax_b = np.abs(ref.y.astype(np.float64)).reshape(R, C // 32, 32).max(axis=2)
    t = amax_b / 6.0
    with np.errstate(divide="ignore"):
        frac = np.where(t > 0, t / 2.0 ** np.floor(np.log2(np.maximum(t, 1e-300))), 1.5)  # in [1, 2)
    near = (frac - 1.0 <= 1e-5) | (2.0 - frac <= 2e-5)
    sdiff = scales != ref.scales
    assert not np.any(sdiff & ~near), f"{what}: {np.count_nonzero(sdiff & ~near)} unexcused scale bytes"
    assert np.all(np.abs(scales.astype(int) - ref.scales.astype(int))[sdiff] == 1), f"{what}: excused scale not adjacent"
    got, want = canon_zero(unpack(codes)), canon_zero(unpack(ref.codes))
    cdiff = (got != want) & ~np.repeat(sdiff, 32, axis=1)
    excused = 0
    for r, c in np.argwhere(cdiff):
        v = float(np.float32(ref.y[r, c]) * oracle.mx_block_encode_scale(int(ref.scales[r, c // 32])))
        a = min(abs(v), 6.0)
        if rounding == oracle.RNE:
            thr = E2M1_MIDPOINTS
            step = 0.5 if a < 2 else (1.0 if a < 4 else 2.0)
        else:
            sr_, sc_ = (c, r) if colwise else (r, c)
            u = oracle.sr_draw(seed, sr_offset, sr_ * x_bits.shape[1] + sc_)
            lo = E2M1_GRID[E2M1_GRID <= a].max()
            hi = E2M1_GRID[E2M1_GRID > a].min() if a < 6 else 6.0
            step = max(hi - lo, 0.5)
            thr = np.array([lo + (hi - lo) * (u + 0.5) / 256])
        assert np.min(np.abs(thr - a)) <= 1e-5 * max(a, step), f"{what}: code at {(r, c)} differs away from a threshold (v={v})"
        assert abs(int(got[r, c] & 7) - int(want[r, c] & 7)) <= 1, f"{what}: excused code not adjacent"
        excused += 1
    assert excused + int(np.count_nonzero(sdiff)) * 32 <= max(1e-3 * R * C, 32), f"{what}: too many excused items"
    return {"excused_codes": excused, "excused_scales": int(np.count_nonzero(sdiff)), "elements": R * C}
