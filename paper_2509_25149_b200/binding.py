"""ctypes binding of the C ABI declared in ``include/nvfp4.h``.

Argument marshalling only: every function here passes device pointers of torch tensors (torch is used
for device memory and streams) straight to the C entry point of the same name.  There is no CPU or
PyTorch fallback: if the CUDA library is missing and cannot be built, loading fails loudly.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

OK = 0
ROUND_NEAREST_EVEN, ROUND_STOCHASTIC = 0, 1
SF_LINEAR, SF_SWIZZLED = 0, 1
SR_INDEPENDENT_COPIES, AMAX_PROVIDED, INPUT_FP32, LINEAR_ROW_SCALES = 1, 2, 4, 8
FORMAT_NVFP4, FORMAT_MXFP4, FORMAT_NVFP4_ROWSCALE = 0, 1, 2

EXPORTED = (
    "nvfp4_quantize", "nvfp4_gemm", "nvfp4_linear_fwd_workspace_bytes", "nvfp4_linear_bwd_workspace_bytes",
    "nvfp4_linear_fwd", "nvfp4_linear_bwd", "nvfp4_dequantize", "nvfp4_rht16", "nvfp4_e2m1_sr", "nvfp4_test_wait_timeout", "nvfp4_device_status",
    "nvfp4_set_gemm_tile_n", "nvfp4_set_gemm_experiment", "nvfp4_status_string", "nvfp4_launch_count",
    "nvfp4_linear_fwd_noalloc", "nvfp4_linear_fwd_noalloc_max_bytes",
    "nvfp4_gemm_bf16", "nvfp4_linear_bf16_fwd", "nvfp4_linear_bf16_bwd", "nvfp4_quant_error", "nvfp4_sq_error",
)


class CTensor(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("global_", ctypes.c_void_p),
                ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("sf_layout", ctypes.c_int32),
                ("format", ctypes.c_int32)]


class CQuantOpts(ctypes.Structure):
    _fields_ = [("block_rows", ctypes.c_int32), ("rounding", ctypes.c_int32), ("rht_rowwise", ctypes.c_int32),
                ("rht_colwise", ctypes.c_int32), ("rht_sign_mask", ctypes.c_uint32), ("flags", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("sr_offset", ctypes.c_uint64), ("rht_dim", ctypes.c_int32),
                ("rht_sign_mask_ext", ctypes.c_uint32 * 3)]


class NVFP4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if the in-tree library is missing or stale) the C-ABI library."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        c = ctypes
        vp, i64, i32, u32 = c.c_void_p, c.c_int64, c.c_int32, c.c_uint32
        TP, OP = c.POINTER(CTensor), c.POINTER(CQuantOpts)
        L.nvfp4_quantize.restype, L.nvfp4_quantize.argtypes = i32, [vp, i64, i64, i64, OP, TP, TP, vp]
        L.nvfp4_gemm.restype, L.nvfp4_gemm.argtypes = i32, [TP, TP, vp, i32, i64, i32, vp]
        L.nvfp4_linear_fwd_workspace_bytes.restype = c.c_size_t
        L.nvfp4_linear_fwd_workspace_bytes.argtypes = [i64, i64]
        L.nvfp4_linear_bwd_workspace_bytes.restype = c.c_size_t
        L.nvfp4_linear_bwd_workspace_bytes.argtypes = [i64, i64]
        L.nvfp4_linear_fwd.restype = i32
        L.nvfp4_linear_fwd.argtypes = [vp, vp, i64, i64, i64, OP, vp, TP, TP, TP, i32, vp, c.c_size_t, vp]
        L.nvfp4_linear_fwd_noalloc.restype = i32
        L.nvfp4_linear_fwd_noalloc.argtypes = [vp, vp, i64, i64, i64, OP, vp, TP, TP, TP, i32, vp]
        L.nvfp4_linear_fwd_noalloc_max_bytes.restype, L.nvfp4_linear_fwd_noalloc_max_bytes.argtypes = c.c_size_t, []
        L.nvfp4_linear_bwd.restype = i32
        L.nvfp4_linear_bwd.argtypes = [vp, TP, TP, i64, i64, i64, OP, vp, vp, i32, vp, c.c_size_t, vp]
        L.nvfp4_gemm_bf16.restype = i32
        L.nvfp4_gemm_bf16.argtypes = [vp, i32, i64, vp, i32, i64, i64, i64, i64, vp, i32, i64, i32, vp]
        L.nvfp4_linear_bf16_fwd.restype, L.nvfp4_linear_bf16_fwd.argtypes = i32, [vp, vp, i64, i64, i64, vp, vp]
        L.nvfp4_linear_bf16_bwd.restype = i32
        L.nvfp4_linear_bf16_bwd.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, i32, vp]
        L.nvfp4_quant_error.restype, L.nvfp4_quant_error.argtypes = i32, [vp, i64, i64, i64, TP, vp, vp]
        L.nvfp4_sq_error.restype = i32
        L.nvfp4_sq_error.argtypes = [vp, i32, i64, vp, i32, i64, i64, i64, vp, vp]
        L.nvfp4_dequantize.restype, L.nvfp4_dequantize.argtypes = i32, [TP, vp, vp]
        L.nvfp4_rht16.restype, L.nvfp4_rht16.argtypes = i32, [vp, i64, i64, i64, i32, u32, vp, vp]
        L.nvfp4_e2m1_sr.restype, L.nvfp4_e2m1_sr.argtypes = i32, [vp, vp, i64, vp, vp]
        L.nvfp4_test_wait_timeout.restype, L.nvfp4_test_wait_timeout.argtypes = i32, [ctypes.c_uint64, vp]
        L.nvfp4_device_status.restype, L.nvfp4_device_status.argtypes = i32, [vp, c.POINTER(u32)]
        L.nvfp4_set_gemm_tile_n.restype, L.nvfp4_set_gemm_tile_n.argtypes = i32, [i32]
        L.nvfp4_set_gemm_experiment.restype, L.nvfp4_set_gemm_experiment.argtypes = i32, [i32, i32, vp]
        L.nvfp4_status_string.restype, L.nvfp4_status_string.argtypes = c.c_char_p, [i32]
        L.nvfp4_launch_count.restype, L.nvfp4_launch_count.argtypes = c.c_uint64, []
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().nvfp4_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise NVFP4Error(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


@dataclass
class NVFP4Tensor:
    """Device buffers of one quantized copy ([rows x cols], cols = contraction dimension)."""
    codes: torch.Tensor   # uint8 [rows, cols/2]
    scales: torch.Tensor  # uint8 [rows * cols/16] (linear: viewable as [rows, cols/16])
    glob: torch.Tensor    # float32 [2] = {amax, s_dec}
    rows: int
    cols: int
    sf_layout: int = SF_SWIZZLED
    format: int = FORMAT_NVFP4  # FORMAT_MXFP4: scales are rows * cols/32 UE8M0 bytes, glob unused ({0, 1})

    def c(self) -> CTensor:
        return CTensor(self.codes.data_ptr(), self.scales.data_ptr(), self.glob.data_ptr(), self.rows, self.cols,
                       self.sf_layout, self.format)


def alloc_tensor(rows: int, cols: int, sf_layout: int = SF_SWIZZLED, device="cuda",
                 format: int = FORMAT_NVFP4) -> NVFP4Tensor:
    block = 32 if format == FORMAT_MXFP4 else 16
    glob = torch.zeros((2 * rows if format == FORMAT_NVFP4_ROWSCALE else 2,), dtype=torch.float32, device=device)
    if format == FORMAT_MXFP4:
        glob[1] = 1.0
    return NVFP4Tensor(torch.empty((rows, cols // 2), dtype=torch.uint8, device=device),
                       torch.empty((rows * cols // block,), dtype=torch.uint8, device=device),
                       glob, rows, cols, sf_layout, format)


def quant_opts(block_rows=1, rounding=ROUND_NEAREST_EVEN, rht_rowwise=False, rht_colwise=False, rht_sign_mask=0,
               flags=0, seed=0, sr_offset=0, rht_dim=0) -> CQuantOpts:
    """rht_sign_mask: up to 128 sign bits (bit j negates input j of a chunk); rht_dim: 0 = the format's own size."""
    ext = (ctypes.c_uint32 * 3)(*[(rht_sign_mask >> (32 * i)) & 0xFFFFFFFF for i in (1, 2, 3)])
    return CQuantOpts(block_rows, rounding, int(rht_rowwise), int(rht_colwise), rht_sign_mask & 0xFFFFFFFF, flags, seed,
                      sr_offset, rht_dim, ext)


def _ref(t: Optional[NVFP4Tensor]):
    return ctypes.byref(t.c()) if t is not None else None


def nvfp4_quantize(x: torch.Tensor, opts: CQuantOpts, rowwise: Optional[NVFP4Tensor] = None,
                   colwise: Optional[NVFP4Tensor] = None) -> None:
    assert x.is_cuda and x.dtype in (torch.bfloat16, torch.float32) and x.dim() == 2 and x.stride(1) == 1
    if x.dtype == torch.float32 and not (opts.flags & INPUT_FP32):  # a binary32 source is announced by a flag
        opts = CQuantOpts(opts.block_rows, opts.rounding, opts.rht_rowwise, opts.rht_colwise, opts.rht_sign_mask,
                          opts.flags | INPUT_FP32, opts.seed, opts.sr_offset, opts.rht_dim, opts.rht_sign_mask_ext)
    assert (x.dtype == torch.float32) == bool(opts.flags & INPUT_FP32)
    _check(lib().nvfp4_quantize(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0), ctypes.byref(opts), _ref(rowwise),
                                _ref(colwise), _stream()), "nvfp4_quantize")


def nvfp4_gemm(A: NVFP4Tensor, B: NVFP4Tensor, D: torch.Tensor, accumulate: bool = False) -> None:
    assert D.is_cuda and D.dim() == 2 and D.stride(1) == 1 and D.dtype in (torch.bfloat16, torch.float32)
    _check(lib().nvfp4_gemm(_ref(A), _ref(B), D.data_ptr(), int(D.dtype == torch.float32), D.stride(0),
                            int(accumulate), _stream()), "nvfp4_gemm")


def nvfp4_linear_fwd_workspace_bytes(M: int, K: int) -> int:
    return int(lib().nvfp4_linear_fwd_workspace_bytes(M, K))


def nvfp4_linear_bwd_workspace_bytes(M: int, N: int) -> int:
    return int(lib().nvfp4_linear_bwd_workspace_bytes(M, N))


def nvfp4_linear_fwd(X: torch.Tensor, W: Optional[torch.Tensor], opts: CQuantOpts, Y: torch.Tensor,
                     X_col_saved: Optional[NVFP4Tensor], W_row: NVFP4Tensor, W_col_saved: Optional[NVFP4Tensor],
                     w_is_cached: bool, workspace: torch.Tensor) -> None:
    M, K = X.shape
    N = W_row.rows
    assert X.is_contiguous() and Y.is_contiguous() and Y.dtype == torch.bfloat16 and tuple(Y.shape) == (M, N)
    assert W is None or (W.is_contiguous() and tuple(W.shape) == (N, K))
    _check(lib().nvfp4_linear_fwd(X.data_ptr(), W.data_ptr() if W is not None else None, M, N, K, ctypes.byref(opts),
                                  Y.data_ptr(), _ref(X_col_saved), _ref(W_row), _ref(W_col_saved), int(w_is_cached),
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "nvfp4_linear_fwd")


def nvfp4_linear_fwd_noalloc_max_bytes() -> int:
    return int(lib().nvfp4_linear_fwd_noalloc_max_bytes())


def nvfp4_linear_fwd_noalloc(X: torch.Tensor, W: Optional[torch.Tensor], opts: CQuantOpts, Y: torch.Tensor,
                             X_col_saved: Optional[NVFP4Tensor], W_row: NVFP4Tensor,
                             W_col_saved: Optional[NVFP4Tensor], w_is_cached: bool) -> None:
    """Forward pass for callers that cannot allocate device memory: same as nvfp4_linear_fwd, but the scratch copy
    of X sits in an array built into the library (16 MiB limit; calls must not overlap on the GPU)."""
    M, K = X.shape
    N = W_row.rows
    assert X.is_contiguous() and Y.is_contiguous() and Y.dtype == torch.bfloat16 and tuple(Y.shape) == (M, N)
    assert W is None or (W.is_contiguous() and tuple(W.shape) == (N, K))
    _check(lib().nvfp4_linear_fwd_noalloc(X.data_ptr(), W.data_ptr() if W is not None else None, M, N, K,
                                          ctypes.byref(opts), Y.data_ptr(), _ref(X_col_saved), _ref(W_row),
                                          _ref(W_col_saved), int(w_is_cached), _stream()),
           "nvfp4_linear_fwd_noalloc")


def nvfp4_linear_bwd(dY: torch.Tensor, X_col_saved: Optional[NVFP4Tensor], W_col_saved: Optional[NVFP4Tensor], K: int,
                     opts: CQuantOpts, dX: Optional[torch.Tensor], dW: Optional[torch.Tensor], accumulate_dw: bool,
                     workspace: torch.Tensor) -> None:
    M, N = dY.shape
    assert dY.is_contiguous()
    assert dX is None or (dX.is_contiguous() and dX.dtype == torch.bfloat16 and tuple(dX.shape) == (M, K))
    assert dW is None or (dW.is_contiguous() and dW.dtype == torch.float32 and tuple(dW.shape) == (N, K))
    _check(lib().nvfp4_linear_bwd(dY.data_ptr(), _ref(X_col_saved), _ref(W_col_saved), M, N, K, ctypes.byref(opts),
                                  dX.data_ptr() if dX is not None else None,
                                  dW.data_ptr() if dW is not None else None, int(accumulate_dw),
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()),
           "nvfp4_linear_bwd")


K_MAJOR, MN_MAJOR = 0, 1


def nvfp4_gemm_bf16(A: torch.Tensor, B: torch.Tensor, D: torch.Tensor, a_layout: int = K_MAJOR,
                    b_layout: int = K_MAJOR, accumulate: bool = False) -> None:
    """D[M x N] = op(A) op(B)^T in BF16.  K_MAJOR: the operand is [M or N][K]; MN_MAJOR: it is [K][M or N]."""
    for t in (A, B):
        assert t.is_cuda and t.dim() == 2 and t.stride(1) == 1 and t.dtype == torch.bfloat16
    assert D.is_cuda and D.dim() == 2 and D.stride(1) == 1 and D.dtype in (torch.bfloat16, torch.float32)
    M, N = D.shape
    K = A.shape[0] if a_layout == MN_MAJOR else A.shape[1]
    assert tuple(A.shape) == ((K, M) if a_layout == MN_MAJOR else (M, K))
    assert tuple(B.shape) == ((K, N) if b_layout == MN_MAJOR else (N, K))
    _check(lib().nvfp4_gemm_bf16(A.data_ptr(), a_layout, A.stride(0), B.data_ptr(), b_layout, B.stride(0), M, N, K,
                                 D.data_ptr(), int(D.dtype == torch.float32), D.stride(0), int(accumulate), _stream()),
           "nvfp4_gemm_bf16")


def nvfp4_linear_bf16_fwd(X: torch.Tensor, W: torch.Tensor, Y: torch.Tensor) -> None:
    M, K = X.shape
    N = W.shape[0]
    assert X.is_contiguous() and W.is_contiguous() and Y.is_contiguous() and tuple(W.shape) == (N, K)
    assert X.dtype == W.dtype == Y.dtype == torch.bfloat16 and tuple(Y.shape) == (M, N)
    _check(lib().nvfp4_linear_bf16_fwd(X.data_ptr(), W.data_ptr(), M, N, K, Y.data_ptr(), _stream()),
           "nvfp4_linear_bf16_fwd")


def nvfp4_linear_bf16_bwd(dY: torch.Tensor, X: Optional[torch.Tensor], W: Optional[torch.Tensor], K: int,
                          dX: Optional[torch.Tensor], dW: Optional[torch.Tensor], accumulate_dw: bool = False) -> None:
    M, N = dY.shape
    assert dY.is_contiguous() and dY.dtype == torch.bfloat16
    assert dX is None or (W is not None and W.is_contiguous() and tuple(W.shape) == (N, K) and dX.is_contiguous()
                          and dX.dtype == torch.bfloat16 and tuple(dX.shape) == (M, K))
    assert dW is None or (X is not None and X.is_contiguous() and tuple(X.shape) == (M, K) and dW.is_contiguous()
                          and dW.dtype == torch.float32 and tuple(dW.shape) == (N, K))
    _check(lib().nvfp4_linear_bf16_bwd(dY.data_ptr(), X.data_ptr() if X is not None else None,
                                       W.data_ptr() if W is not None else None, M, N, K,
                                       dX.data_ptr() if dX is not None else None,
                                       dW.data_ptr() if dW is not None else None, int(accumulate_dw), _stream()),
           "nvfp4_linear_bf16_bwd")


def nvfp4_quant_error(x: torch.Tensor, q: NVFP4Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Device tensor {sum (x - decode(q))^2, sum x^2} (float64) for the row-wise copy q of x."""
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1 and x.dtype == torch.bfloat16
    out = torch.empty(2, dtype=torch.float64, device=x.device) if out is None else out
    _check(lib().nvfp4_quant_error(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0), _ref(q), out.data_ptr(),
                                   _stream()), "nvfp4_quant_error")
    return out


def nvfp4_sq_error(ref: torch.Tensor, test: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Device tensor {sum (ref - test)^2, sum ref^2} (float64) of two 2-D tensors, each bf16 or fp32."""
    for t in (ref, test):
        assert t.is_cuda and t.dim() == 2 and t.stride(1) == 1 and t.dtype in (torch.bfloat16, torch.float32)
    assert ref.shape == test.shape
    out = torch.empty(2, dtype=torch.float64, device=ref.device) if out is None else out
    _check(lib().nvfp4_sq_error(ref.data_ptr(), int(ref.dtype == torch.float32), ref.stride(0), test.data_ptr(),
                                int(test.dtype == torch.float32), test.stride(0), ref.shape[0], ref.shape[1],
                                out.data_ptr(), _stream()), "nvfp4_sq_error")
    return out


def nvfp4_dequantize(t: NVFP4Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    if out is None:
        out = torch.empty((t.rows, t.cols), dtype=torch.float32, device=t.codes.device)
    _check(lib().nvfp4_dequantize(_ref(t), out.data_ptr(), _stream()), "nvfp4_dequantize")
    return out


def nvfp4_rht16(x: torch.Tensor, colwise: bool, sign_mask: int) -> torch.Tensor:
    R, C = (x.shape[1], x.shape[0]) if colwise else tuple(x.shape)
    out = torch.empty((R, C), dtype=torch.float32, device=x.device)
    _check(lib().nvfp4_rht16(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0), int(colwise), sign_mask,
                             out.data_ptr(), _stream()), "nvfp4_rht16")
    return out


def nvfp4_e2m1_sr(v: torch.Tensor, u: torch.Tensor) -> torch.Tensor:
    """E2M1 codes of the scaled fp32 values `v` under stochastic rounding with the uint8 draws `u` (test aid)."""
    assert v.dtype == torch.float32 and u.dtype == torch.uint8 and v.numel() == u.numel()
    v, u = v.contiguous(), u.contiguous()
    out = torch.empty(v.numel(), dtype=torch.uint8, device=v.device)
    _check(lib().nvfp4_e2m1_sr(v.data_ptr(), u.data_ptr(), v.numel(), out.data_ptr(), _stream()), "nvfp4_e2m1_sr")
    return out


def nvfp4_test_wait_timeout(limit_ns: int) -> None:
    """Enqueues the test kernel whose bounded wait runs out after `limit_ns` (the status word then holds 0x7E570001)."""
    _check(lib().nvfp4_test_wait_timeout(limit_ns, _stream()), "nvfp4_test_wait_timeout")


def nvfp4_device_status() -> int:
    """Synchronises the current stream; raises if a bounded device-side wait expired."""
    detail = ctypes.c_uint32(0)
    st = lib().nvfp4_device_status(_stream(), ctypes.byref(detail))
    if st != OK:
        raise NVFP4Error(st, f"nvfp4_device_status (code 0x{detail.value:x})")
    return 0


def nvfp4_set_gemm_experiment(mode: int = 0, max_pairs: int = 0, probe: Optional[torch.Tensor] = None) -> None:
    """Measurement aid of the CTA-pair GEMM (see the header); probe: int64 device tensor of 8 words per pair."""
    assert probe is None or (probe.dtype == torch.int64 and probe.is_contiguous())
    if lib().nvfp4_set_gemm_experiment(mode, max_pairs, probe.data_ptr() if probe is not None else None) != 0:
        raise ValueError("nvfp4_set_gemm_experiment: value out of range")


def nvfp4_set_gemm_tile_n(tile_n: int) -> None:
    if lib().nvfp4_set_gemm_tile_n(tile_n) != 0:
        raise ValueError("tile_n must be 0, 128, 256 or 512")


def nvfp4_launch_count() -> int:
    return int(lib().nvfp4_launch_count())
