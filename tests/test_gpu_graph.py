"""The composed calls are stream-ordered and allocation-free, so a step can be captured in a CUDA graph and replayed;
the replay must reproduce the direct calls bit for bit (the kernels are deterministic)."""
import pytest
import torch

from paper_2509_25149_b200 import binding as B
from paper_2509_25149_b200 import synth

pytestmark = pytest.mark.gpu


def test_captured_step_replays_bit_for_bit():
    M, N, K = 1024, 1536, 768
    g = torch.Generator(device="cuda").manual_seed(7)
    X = torch.randn((M, K), generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    dY = (torch.randn((M, N), generator=g, device="cuda") * 1e-3).to(torch.bfloat16)
    opts = B.quant_opts(rht_sign_mask=synth.DEFAULT_RHT_SIGN_MASK, seed=3, sr_offset=5)
    X_col, W_row, W_col = B.alloc_tensor(K, M), B.alloc_tensor(N, K), B.alloc_tensor(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")

    def step():
        B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
        B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, dW, False, ws_b)

    step()  # first call outside the capture: it sets kernel attributes and fills the tensor-map cache
    torch.cuda.synchronize()
    B.nvfp4_device_status()
    want = [t.clone() for t in (Y, dX, dW, W_row.codes, W_col.codes, X_col.codes, W_row.glob, X_col.glob)]

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for t in (Y, dX, dW, W_row.codes, W_col.codes, X_col.codes):
        t.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    B.nvfp4_device_status()
    for got, ref in zip((Y, dX, dW, W_row.codes, W_col.codes, X_col.codes, W_row.glob, X_col.glob), want):
        assert torch.equal(got, ref)
