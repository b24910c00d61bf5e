"""CPU oracle for the NVFP4 quantize + block-scaled GEMM path.

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in ``nvfp4_oracle.c`` (plain C,
binary32 steps written one rounding at a time, binary64 for every reference
quantity); this module compiles it with gcc and exposes it through ctypes on
numpy arrays.  It shares nothing with the CUDA path and must never be imported
by the product package.

Functions follow the paper's Appendix B (Eq. 1-5), Appendix C (random Hadamard
transform), Section 4.3 (2D weight blocks) and Section 4.4 (stochastic
rounding); each C function cites the passage it restates.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "nvfp4_oracle.c")
_LIB = os.path.join(_DIR, "libnvfp4_oracle.so")
_lock = threading.Lock()
_lib = None

RNE, SR = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle (strict IEEE: no contraction, no fast-math)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-fvisibility=hidden", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            c = ctypes
            u8p, u16p, u32p = c.POINTER(c.c_uint8), c.POINTER(c.c_uint16), c.POINTER(c.c_uint32)
            f32p, f64p = c.POINTER(c.c_float), c.POINTER(c.c_double)
            sig = {
                "orc_bf16_to_f32": (c.c_float, [c.c_uint16]),
                "orc_e2m1_decode": (c.c_float, [c.c_uint8]),
                "orc_e4m3_decode": (c.c_float, [c.c_uint8]),
                "orc_e4m3_encode_rne": (c.c_uint8, [c.c_float]),
                "orc_e2m1_encode_rne": (c.c_uint8, [c.c_float]),
                "orc_e2m1_encode_sr": (c.c_uint8, [c.c_float, c.c_uint8]),
                "orc_e2m1_encode_sr_many": (None, [f32p, u8p, c.c_int64, u8p]),
                "orc_philox4x32_10": (None, [u32p, u32p, u32p]),
                "orc_sr_draw": (c.c_uint8, [c.c_uint64, c.c_uint64, c.c_uint64]),
                "orc_hadamard16_entry": (c.c_int, [c.c_int, c.c_int]),
                "orc_rht16": (None, [f32p, c.c_uint16, f32p]),
                "orc_global_scale": (None, [c.c_float, f32p, f32p]),
                "orc_block_scale_byte": (c.c_uint8, [c.c_float, c.c_float]),
                "orc_block_encode_scale": (c.c_float, [c.c_uint8, c.c_float]),
                "orc_sf_swizzled_offset": (c.c_int64, [c.c_int64, c.c_int64, c.c_int64]),
                "orc_quantize": (c.c_int, [u16p, c.c_int64, c.c_int64, c.c_int64, c.c_int, c.c_int,
                                           c.c_int, c.c_uint16, c.c_int, c.c_uint64, c.c_uint64,
                                           c.c_float, c.c_int64, c.c_int64, c.c_int64, u8p, u8p, f32p, f32p]),
                "orc_quantize_f32": (c.c_int, [f32p, c.c_int64, c.c_int64, c.c_int64, c.c_int, c.c_int,
                                               c.c_int, c.c_uint16, c.c_int, c.c_uint64, c.c_uint64,
                                               c.c_float, c.c_int64, c.c_int64, c.c_int64, u8p, u8p, f32p, f32p]),
                "orc_rht_d": (c.c_int, [f32p, c.c_int, u32p, f32p]),
                "orc_quantize_rht": (c.c_int, [u16p, c.c_int64, c.c_int64, c.c_int64, c.c_int, c.c_int, u32p,
                                               c.c_int, c.c_uint64, c.c_uint64, c.c_float, c.c_int64, c.c_int64,
                                               c.c_int64, u8p, u8p, f32p, f32p]),
                "orc_dequantize": (None, [u8p, u8p, f32p, c.c_int64, c.c_int64, f64p]),
                "orc_dequantize_local": (None, [u8p, u8p, c.c_int64, c.c_int64, f64p]),
                "orc_gemm_tn": (None, [f64p, f64p, c.c_int64, c.c_int64, c.c_int64, f64p, f64p]),
                "orc_gemm_blockscaled": (None, [u8p, u8p, f32p, u8p, u8p, f32p, c.c_int64,
                                                c.c_int64, c.c_int64, f64p]),
                "orc_ue8m0_decode": (c.c_float, [c.c_uint8]),
                "orc_mx_block_scale_byte": (c.c_uint8, [c.c_float]),
                "orc_mx_block_encode_scale": (c.c_float, [c.c_uint8]),
                "orc_hadamard32_entry": (c.c_int, [c.c_int, c.c_int]),
                "orc_rht32": (None, [f32p, c.c_uint32, f32p]),
                "orc_quantize_mx": (c.c_int, [u16p, c.c_int64, c.c_int64, c.c_int64, c.c_int, c.c_int,
                                              c.c_int, c.c_uint32, c.c_int, c.c_uint64, c.c_uint64,
                                              c.c_int64, c.c_int64, c.c_int64, u8p, u8p, f32p]),
                "orc_dequantize_mx": (None, [u8p, u8p, c.c_int64, c.c_int64, f64p]),
            }
            for name, (res, args) in sig.items():
                fn = getattr(L, name)
                fn.restype, fn.argtypes = res, args
            _lib = L
    return _lib


def _p(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


# ---------------------------------------------------------------- scalars ----
def bf16_to_f32(h: int) -> float:
    return float(lib().orc_bf16_to_f32(h))


def e2m1_decode(code: int) -> float:
    return float(lib().orc_e2m1_decode(code))


def e4m3_decode(byte: int) -> float:
    return float(lib().orc_e4m3_decode(byte))


def e4m3_encode_rne(t: float) -> int:
    return int(lib().orc_e4m3_encode_rne(np.float32(t)))


def e2m1_encode_rne(v: float) -> int:
    return int(lib().orc_e2m1_encode_rne(np.float32(v)))


def e2m1_encode_sr(v: float, u: int) -> int:
    return int(lib().orc_e2m1_encode_sr(np.float32(v), u))


def e2m1_encode_sr_many(v, u):
    """orc_e2m1_encode_sr applied element by element to float32 values `v` and uint8 draws `u`."""
    v = np.ascontiguousarray(v, dtype=np.float32).ravel()
    u = np.ascontiguousarray(u, dtype=np.uint8).ravel()
    assert v.size == u.size
    out = np.empty(v.size, dtype=np.uint8)
    lib().orc_e2m1_encode_sr_many(_p(v, ctypes.c_float), _p(u, ctypes.c_uint8), v.size, _p(out, ctypes.c_uint8))
    return out


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32), _p(out, ctypes.c_uint32))
    return out


def sr_draw(seed: int, sr_offset: int, e: int) -> int:
    return int(lib().orc_sr_draw(seed, sr_offset, e))


def hadamard16_entry(j: int, k: int) -> int:
    return int(lib().orc_hadamard16_entry(j, k))


def rht16(x, sign_mask: int):
    xin = np.ascontiguousarray(x, dtype=np.float32)
    assert xin.shape == (16,)
    y = np.zeros(16, dtype=np.float32)
    lib().orc_rht16(_p(xin, ctypes.c_float), sign_mask, _p(y, ctypes.c_float))
    return y


def _sign_words(sign_mask: int):
    return np.array([(sign_mask >> (32 * i)) & 0xFFFFFFFF for i in range(4)], dtype=np.uint32)


def rht_d(x, d: int, sign_mask: int):
    """Transform of size d (a power of two up to 128) of one chunk; bit j of sign_mask negates input j."""
    xin = np.ascontiguousarray(x, dtype=np.float32)
    assert xin.shape == (d,)
    y = np.zeros(d, dtype=np.float32)
    w = _sign_words(sign_mask)
    if lib().orc_rht_d(_p(xin, ctypes.c_float), d, _p(w, ctypes.c_uint32), _p(y, ctypes.c_float)) != 0:
        raise ValueError("transform size must be a power of two in [2, 128]")
    return y


def global_scale(amax: float):
    e, d = ctypes.c_float(), ctypes.c_float()
    lib().orc_global_scale(np.float32(amax), ctypes.byref(e), ctypes.byref(d))
    return np.float32(e.value), np.float32(d.value)


def block_scale_byte(amax_b: float, s_enc: float) -> int:
    return int(lib().orc_block_scale_byte(np.float32(amax_b), np.float32(s_enc)))


def block_encode_scale(scale_byte: int, s_dec: float):
    return np.float32(lib().orc_block_encode_scale(scale_byte, np.float32(s_dec)))


def sf_swizzled_offset(r: int, kb: int, n_kb: int) -> int:
    return int(lib().orc_sf_swizzled_offset(r, kb, n_kb))


def sf_unswizzle(swizzled, rows: int, n_kb: int):
    """Gather a swizzled scale buffer back into the linear [rows][n_kb] layout."""
    flat = np.asarray(swizzled, dtype=np.uint8).reshape(-1)
    r = np.arange(rows, dtype=np.int64)[:, None]
    kb = np.arange(n_kb, dtype=np.int64)[None, :]
    off = ((r // 128) * (n_kb // 4) + kb // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4
    return flat[off]


def sf_swizzle(linear):
    """Scatter a linear [rows][n_kb] scale array into the swizzled byte order (rows % 128 == 0, n_kb % 4 == 0)."""
    lin = np.asarray(linear, dtype=np.uint8)
    rows, n_kb = lin.shape
    r = np.arange(rows, dtype=np.int64)[:, None]
    kb = np.arange(n_kb, dtype=np.int64)[None, :]
    off = ((r // 128) * (n_kb // 4) + kb // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4
    out = np.zeros(rows * n_kb, dtype=np.uint8)
    out[off.reshape(-1)] = lin.reshape(-1)
    return out


# ---------------------------------------------------------------- tensors ----
class Quantized:
    """One NVFP4 copy: codes [R][C/2], scales [R][C/16] (linear), global {amax, s_dec}."""

    def __init__(self, codes, scales, glob, rows, cols, y=None):
        self.codes, self.scales, self.glob = codes, scales, glob
        self.rows, self.cols, self.y = rows, cols, y

    @property
    def amax(self):
        return self.glob[0]

    @property
    def s_dec(self):
        return self.glob[1]


def quantize(x_bf16_bits, *, colwise=False, block_rows=1, rht=False, sign_mask=0, rounding=RNE,
             seed=0, sr_offset=0, amax_override=None, return_y=False, sr_row0=0, sr_cols=0, sr_col0=0,
             rht_dim=16) -> Quantized:
    """Quantize one copy of a bf16 tensor given as a 2-D uint16 array of bit patterns (or of a binary32 tensor given
    as a float32 array).

    sr_row0 / sr_col0 / sr_cols: the array is the block starting at (sr_row0, sr_col0) of a larger source with
    sr_cols columns (only the index of the stochastic-rounding draws depends on it).
    rht_dim: size of the transform when rht is set (16 = the recipe; 2, 4, 8, 128 = the sizes of Appendix E.4.2,
    bf16 sources with 1x16 blocks only); sign_mask then carries rht_dim bits."""
    x = np.asarray(x_bf16_bits)
    f32 = x.dtype == np.float32  # a binary32 source instead of bf16 bit patterns
    assert (x.dtype == np.uint16 or f32) and x.ndim == 2
    esz = 4 if f32 else 2
    ld = x.strides[0] // esz
    assert x.strides[1] == esz
    sr, sc = x.shape
    R, C = (sc, sr) if colwise else (sr, sc)
    codes = np.zeros((R, C // 2), dtype=np.uint8)
    scales = np.zeros((R, C // 16), dtype=np.uint8)
    glob = np.zeros(2, dtype=np.float32)
    y = np.zeros((R, C), dtype=np.float32) if return_y else None
    amax_arg = np.float32(-1.0 if amax_override is None else amax_override)
    outs = (_p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8), _p(glob, ctypes.c_float),
            _p(y, ctypes.c_float) if return_y else None)
    if rht and rht_dim != 16:
        if f32 or block_rows != 1:
            raise ValueError("other transform sizes: bf16 source and 1x16 blocks only")
        w = _sign_words(sign_mask)
        rc = lib().orc_quantize_rht(_p(x, ctypes.c_uint16), sr, sc, ld, int(colwise), rht_dim, _p(w, ctypes.c_uint32),
                                    rounding, seed, sr_offset, amax_arg, sr_row0, sr_cols, sr_col0, *outs)
    else:
        fn, src = ((lib().orc_quantize_f32, _p(x, ctypes.c_float)) if f32
                   else (lib().orc_quantize, _p(x, ctypes.c_uint16)))
        rc = fn(src, sr, sc, ld, int(colwise), block_rows, int(rht), sign_mask & 0xFFFF, rounding, seed, sr_offset,
                amax_arg, sr_row0, sr_cols, sr_col0, *outs)
    if rc != 0:
        raise ValueError(f"orc_quantize rejected the shape (rc={rc})")
    return Quantized(codes, scales, glob, R, C, y)


def dequantize(q: Quantized, local_only=False):
    out = np.zeros((q.rows, q.cols), dtype=np.float64)
    codes = np.ascontiguousarray(q.codes)
    scales = np.ascontiguousarray(q.scales)
    if local_only:
        lib().orc_dequantize_local(_p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8), q.rows,
                                   q.cols, _p(out, ctypes.c_double))
    else:
        g = np.ascontiguousarray(q.glob, dtype=np.float32)
        lib().orc_dequantize(_p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8),
                             _p(g, ctypes.c_float), q.rows, q.cols, _p(out, ctypes.c_double))
    return out


def gemm_tn(A, B, want_T=True):
    """D[i,j] = sum_k A[i,k] B[j,k] in binary64 (naive); T = sum |A||B|."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    D = np.zeros((M, N), dtype=np.float64)
    T = np.zeros((M, N), dtype=np.float64) if want_T else None
    lib().orc_gemm_tn(_p(A, ctypes.c_double), _p(B, ctypes.c_double), M, N, K,
                      _p(D, ctypes.c_double), _p(T, ctypes.c_double) if want_T else None)
    return (D, T) if want_T else D


def gemm_blockscaled(a: Quantized, b: Quantized):
    assert a.cols == b.cols
    D = np.zeros((a.rows, b.rows), dtype=np.float64)
    ag = np.ascontiguousarray(a.glob, dtype=np.float32)
    bg = np.ascontiguousarray(b.glob, dtype=np.float32)
    ac, asf = np.ascontiguousarray(a.codes), np.ascontiguousarray(a.scales)
    bc, bsf = np.ascontiguousarray(b.codes), np.ascontiguousarray(b.scales)
    lib().orc_gemm_blockscaled(_p(ac, ctypes.c_uint8), _p(asf, ctypes.c_uint8), _p(ag, ctypes.c_float),
                               _p(bc, ctypes.c_uint8), _p(bsf, ctypes.c_uint8), _p(bg, ctypes.c_float),
                               a.rows, b.rows, a.cols, _p(D, ctypes.c_double))
    return D


# ------------------------- global scale at row granularity (Appendix B.1, last sentence) ----
class QuantizedRows:
    """A row-wise copy whose FP32 scale is taken per row: glob[r] = {amax of row r, s_dec of row r}."""

    def __init__(self, codes, scales, glob, rows, cols):
        self.codes, self.scales, self.glob = codes, scales, glob
        self.rows, self.cols = rows, cols


def quantize_rowscale(x_bf16_bits, *, rounding=RNE, seed=0, sr_offset=0, sr_row0=0, sr_cols=0, sr_col0=0) -> QuantizedRows:
    """Appendix B.1 closes with the remark that the global scale could span a row instead of the tensor, which
    removes the pass that computes the tensor amax.  Written out: every row is quantized as a tensor of its own
    (Eq. 1 from the row's amax, then Eq. 2-4 unchanged); the stochastic-rounding draws stay keyed by the element's
    position in the whole source."""
    x = np.asarray(x_bf16_bits)
    assert x.dtype == np.uint16 and x.ndim == 2
    R, C = x.shape
    codes = np.zeros((R, C // 2), dtype=np.uint8)
    scales = np.zeros((R, C // 16), dtype=np.uint8)
    glob = np.zeros((R, 2), dtype=np.float32)
    for r in range(R):
        q = quantize(x[r:r + 1], rounding=rounding, seed=seed, sr_offset=sr_offset, sr_row0=sr_row0 + r,
                     sr_cols=sr_cols if sr_cols else C, sr_col0=sr_col0)
        codes[r], scales[r], glob[r] = q.codes[0], q.scales[0], q.glob
    return QuantizedRows(codes, scales, glob, R, C)


def dequantize_rowscale(q: QuantizedRows):
    """x^ = code * block scale * the row's decode scale, in binary64."""
    out = np.zeros((q.rows, q.cols), dtype=np.float64)
    for r in range(q.rows):
        out[r] = dequantize(Quantized(q.codes[r:r + 1], q.scales[r:r + 1], q.glob[r], 1, q.cols))[0]
    return out


# ------------------------------------------- layers kept in BF16 (Section 4.1) ----
def _bf16_bits_to_f64(bits):
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def linear_bf16_fwd(x_bits, w_bits):
    """A linear layer left in BF16 (Section 4.1 keeps the most sensitive layers in higher precision; Appendix D
    switches all of them late in training): Y = X W^T of the bf16 values, exact products summed in binary64.
    Returns (Y, T) with T = |X| |W|^T, the scale of the accumulation-error tolerance."""
    return gemm_tn(_bf16_bits_to_f64(x_bits), _bf16_bits_to_f64(w_bits))


def linear_bf16_bwd(dy_bits, x_bits, w_bits):
    """dX = dY W and dW = dY^T X (Section 4.1's Dgrad and Wgrad) of the bf16 values, in binary64.
    Returns ((dX, T_dX), (dW, T_dW))."""
    dy, x, w = _bf16_bits_to_f64(dy_bits), _bf16_bits_to_f64(x_bits), _bf16_bits_to_f64(w_bits)
    return gemm_tn(dy, np.ascontiguousarray(w.T)), gemm_tn(np.ascontiguousarray(dy.T), np.ascontiguousarray(x.T))


# ------------------------------- quantization-error metric (Appendix E.2) ----
def quant_error(x, x_hat):
    """Squared error of a decoded tensor against its source and the source's squared norm, in binary64:
    (sum (x - x_hat)^2, sum x^2); their ratio is the relative quantization error of the tensor."""
    x = np.asarray(x, dtype=np.float64)
    e = x - np.asarray(x_hat, dtype=np.float64)
    return float(np.sum(e * e)), float(np.sum(x * x))


# ----------------------------------------------------------------- MXFP4 ----
def ue8m0_decode(b: int) -> float:
    return float(lib().orc_ue8m0_decode(b))


def mx_block_scale_byte(amax_b: float) -> int:
    return int(lib().orc_mx_block_scale_byte(np.float32(amax_b)))


def mx_block_encode_scale(b: int):
    return np.float32(lib().orc_mx_block_encode_scale(b))


def hadamard32_entry(j: int, k: int) -> int:
    return int(lib().orc_hadamard32_entry(j, k))


def rht32(x, sign_mask: int):
    xin = np.ascontiguousarray(x, dtype=np.float32)
    assert xin.shape == (32,)
    y = np.zeros(32, dtype=np.float32)
    lib().orc_rht32(_p(xin, ctypes.c_float), sign_mask, _p(y, ctypes.c_float))
    return y


class QuantizedMX:
    """One MXFP4 copy: codes [R][C/2], UE8M0 scales [R][C/32] (linear); no tensor-level scale."""

    def __init__(self, codes, scales, rows, cols, y=None):
        self.codes, self.scales = codes, scales
        self.rows, self.cols, self.y = rows, cols, y


def quantize_mx(x_bf16_bits, *, colwise=False, block_rows=1, rht=False, sign_mask=0, rounding=RNE, seed=0,
                sr_offset=0, return_y=False, sr_row0=0, sr_cols=0, sr_col0=0) -> QuantizedMX:
    """MXFP4 quantization of one copy of a bf16 tensor given as a 2-D uint16 array of bit patterns."""
    x = np.asarray(x_bf16_bits)
    assert x.dtype == np.uint16 and x.ndim == 2 and x.strides[1] == 2
    ld = x.strides[0] // 2
    sr, sc = x.shape
    R, C = (sc, sr) if colwise else (sr, sc)
    codes = np.zeros((R, C // 2), dtype=np.uint8)
    scales = np.zeros((R, max(C // 32, 1)), dtype=np.uint8)
    y = np.zeros((R, C), dtype=np.float32) if return_y else None
    rc = lib().orc_quantize_mx(_p(x, ctypes.c_uint16), sr, sc, ld, int(colwise), block_rows, int(rht), sign_mask,
                               rounding, seed, sr_offset, sr_row0, sr_cols, sr_col0, _p(codes, ctypes.c_uint8),
                               _p(scales, ctypes.c_uint8), _p(y, ctypes.c_float) if return_y else None)
    if rc != 0:
        raise ValueError(f"orc_quantize_mx rejected the shape (rc={rc})")
    return QuantizedMX(codes, scales, R, C, y)


def dequantize_mx(q: QuantizedMX):
    out = np.zeros((q.rows, q.cols), dtype=np.float64)
    codes = np.ascontiguousarray(q.codes)
    scales = np.ascontiguousarray(q.scales)
    lib().orc_dequantize_mx(_p(codes, ctypes.c_uint8), _p(scales, ctypes.c_uint8), q.rows, q.cols,
                            _p(out, ctypes.c_double))
    return out
