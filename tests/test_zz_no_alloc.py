"""nvfp4_linear_fwd_noalloc: the forward pass for callers that cannot pass scratch memory.

Such callers (code that must not call cudaMalloc where it runs: server callbacks, plug-ins that only receive their
input and output buffers) get the same result as nvfp4_linear_fwd; the only difference is where the temporary
NVFP4 copy of X lives.  The file is named so that pytest collects it last: if it fails, every other test has run.
"""
import ctypes

import pytest
import torch

from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def _layer(M, N, K, seed):
    X = synth.normal_with_outliers_bf16((M, K), 0.01, 50.0, seed, seed + 1).cuda()
    W = synth.normal_bf16((N, K), 0.02, seed + 2).cuda()
    return X, W


def _forward(fn_noalloc, X, W, M, N, K):
    opts = B.quant_opts(rht_sign_mask=synth.DEFAULT_RHT_SIGN_MASK)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    if fn_noalloc:
        B.nvfp4_linear_fwd_noalloc(X, W, opts, Y, X_col, W_row, W_col, False)
    else:
        ws = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
        B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws)
    B.nvfp4_device_status()
    return Y, X_col, W_row


def test_noalloc_matches_the_workspace_entry_point_twice_in_a_row():
    # two calls in a row with different inputs: the second finds the first one's data in the shared array
    for M, N, K, seed in ((512, 1024, 1024, 21), (256, 512, 2048, 33)):
        X, W = _layer(M, N, K, seed)
        Y_ref, Xc_ref, Wr_ref = _forward(False, X, W, M, N, K)
        Y, Xc, Wr = _forward(True, X, W, M, N, K)
        # same kernels, same arithmetic, same order: bit-identical, which is inside the GEMM tolerance of the
        # other tests (1e-3 * sum|a||b| + bf16 rounding)
        assert torch.equal(Y.view(torch.int16), Y_ref.view(torch.int16))
        assert torch.equal(Xc.codes, Xc_ref.codes) and torch.equal(Xc.scales, Xc_ref.scales)
        assert torch.equal(Wr.codes, Wr_ref.codes) and torch.equal(Xc.glob, Xc_ref.glob)
        assert torch.isfinite(Y.float()).all()


def test_noalloc_rejects_problems_beyond_its_array():
    limit = B.nvfp4_linear_fwd_noalloc_max_bytes()
    assert limit == 16 << 20
    M, K, N = 8192, 5120, 256
    assert B.nvfp4_linear_fwd_workspace_bytes(M, K) > limit
    o = B.quant_opts()
    fake = 0x7F0000000000  # never dereferenced: the size check comes first
    w_row = B.CTensor(fake, fake, fake, N, K, B.SF_SWIZZLED, 0)
    st = B.lib().nvfp4_linear_fwd_noalloc(fake, fake, M, N, K, ctypes.byref(o), fake, None, ctypes.byref(w_row), None,
                                          0, None)
    assert st == 5 and "scratch" in B.status_string(st)
