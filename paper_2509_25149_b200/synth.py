"""Seeded synthetic tensors shaped like the paper's 12B-class linear layers.

This module only draws random numbers and casts them to bf16; it contains none
of the NVFP4 arithmetic, so the CPU oracle's tests and the CUDA path's tests may
both take their inputs from it.

Recipe: torch CPU generator seeded with ``1000 * cfg + tensor_id`` (+ 10 * layer
for multi-layer configs), values drawn in fp32, transformed, rounded to bf16
(round-to-nearest-even).  tensor ids: X = 1, W = 2, dY = 3, outlier mask = 4.
Dimensions follow the 12B model's table (hidden 5120, FFN 20480, 40 query and
8 key-value heads of size 128, squared-ReLU FFN, sequence 8192).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

X_ID, W_ID, DY_ID, MASK_ID = 1, 2, 3, 4
DEFAULT_RHT_SIGN_MASK = 0x73E5  # low 16 bits of Philox4x32-10(key 0, counter (0,0,0,1)) word 0


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def normal_bf16(shape, std: float, seed: int) -> torch.Tensor:
    x = torch.randn(shape, generator=_gen(seed), dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(torch.bfloat16)


def normal_with_outliers_bf16(shape, frac: float, factor: float, seed: int, mask_seed: int) -> torch.Tensor:
    """N(0,1) with a Bernoulli(frac) subset of entries multiplied by ``factor``."""
    x = torch.randn(shape, generator=_gen(seed), dtype=torch.float32)
    m = torch.rand(shape, generator=_gen(mask_seed), dtype=torch.float32) < frac
    x = torch.where(m, x * factor, x)
    return x.to(torch.bfloat16)


def squared_relu_bf16(shape, seed: int) -> torch.Tensor:
    """max(z, 0)^2 with z ~ N(0,1): half zeros, heavy right tail."""
    z = torch.randn(shape, generator=_gen(seed), dtype=torch.float32)
    return torch.clamp_min(z, 0).square_().to(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (CPU) -> uint16 numpy array of its bit patterns (shares memory)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


@dataclass
class LinearProblem:
    """One linear layer: X [M x K], W [N x K], dY [M x N]."""
    name: str
    M: int
    N: int
    K: int
    X: torch.Tensor
    W: torch.Tensor
    dY: torch.Tensor
    sr_seed: int = 0
    sr_offset: int = 0
    rht_sign_mask: int = DEFAULT_RHT_SIGN_MASK


def config1() -> LinearProblem:
    """Small single layer: 512 tokens, 1024 -> 1024, 1% outliers x50."""
    s = 1000
    M, N, K = 512, 1024, 1024
    return LinearProblem("cfg1_linear_512x1024x1024", M, N, K,
                         normal_with_outliers_bf16((M, K), 0.01, 50.0, s + X_ID, s + MASK_ID),
                         normal_bf16((N, K), 0.02, s + W_ID),
                         normal_bf16((M, N), 1e-3, s + DY_ID))


def config2_x() -> torch.Tensor:
    """Quantizer sweep activation: [8192 x 5120] N(0,1), 0.1% outliers x100."""
    s = 2000
    return normal_with_outliers_bf16((8192, 5120), 0.001, 100.0, s + X_ID, s + MASK_ID)


def config2_w() -> torch.Tensor:
    """Quantizer sweep weight: [20480 x 5120] N(0, 0.02)."""
    return normal_bf16((20480, 5120), 0.02, 2000 + W_ID)


def config3(M: int = 8192) -> LinearProblem:
    """FFN up-projection: K = 5120 -> N = 20480."""
    s = 3000
    N, K = 20480, 5120
    return LinearProblem("cfg3_ffn_up_8192x20480x5120", M, N, K,
                         normal_with_outliers_bf16((M, K), 0.001, 100.0, s + X_ID, s + MASK_ID),
                         normal_bf16((N, K), 0.02, s + W_ID),
                         normal_bf16((M, N), 1e-4, s + DY_ID))


def config4(M: int = 8192) -> LinearProblem:
    """FFN down-projection: K = 20480 -> N = 5120, squared-ReLU input."""
    s = 4000
    N, K = 5120, 20480
    return LinearProblem("cfg4_ffn_down_8192x5120x20480", M, N, K,
                         squared_relu_bf16((M, K), s + X_ID),
                         normal_bf16((N, K), 0.01, s + W_ID),
                         normal_bf16((M, N), 1e-4, s + DY_ID))


CONFIG5_LAYERS = (("qkv", 7168, 5120), ("out_proj", 5120, 5120), ("ffn_up", 20480, 5120),
                  ("ffn_down", 5120, 20480))


def config5_layer(layer: int, M: int = 16384) -> LinearProblem:
    """One of the four linears of a transformer block at 16384 tokens."""
    name, N, K = CONFIG5_LAYERS[layer]
    s = 5000 + 10 * layer
    if name == "ffn_down":
        X = squared_relu_bf16((M, K), s + X_ID)
    else:
        X = normal_with_outliers_bf16((M, K), 0.001, 100.0, s + X_ID, s + MASK_ID)
    return LinearProblem(f"cfg5_{name}_{M}x{N}x{K}", M, N, K, X,
                         normal_bf16((N, K), 0.02, s + W_ID),
                         normal_bf16((M, N), 1e-4, s + DY_ID), sr_offset=layer)


# ---------------------------------------------------------------------------------------------
# The same distributions drawn ON THE DEVICE, in row chunks (for the largest configs, where drawing on the host
# would dominate a test): torch CUDA generator seeded like the host recipe.  The values differ from the host
# recipe's (another generator); tests that use these read back the slabs they hand to the oracle.
# ---------------------------------------------------------------------------------------------
def _device_tensor(shape, seed: int, make, device="cuda", chunk_rows: int = 4096) -> torch.Tensor:
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    g = torch.Generator(device=device).manual_seed(seed)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        out[r0:r1] = make((r1 - r0, shape[1]), g).to(torch.bfloat16)
    return out


def normal_bf16_device(shape, std: float, seed: int, device="cuda") -> torch.Tensor:
    return _device_tensor(shape, seed, lambda sh, g: torch.randn(sh, generator=g, device=device) * std, device)


def normal_with_outliers_bf16_device(shape, frac: float, factor: float, seed: int, device="cuda") -> torch.Tensor:
    def make(sh, g):
        x = torch.randn(sh, generator=g, device=device)
        return torch.where(torch.rand(sh, generator=g, device=device) < frac, x * factor, x)
    return _device_tensor(shape, seed, make, device)


def squared_relu_bf16_device(shape, seed: int, device="cuda") -> torch.Tensor:
    return _device_tensor(shape, seed, lambda sh, g: torch.clamp_min(torch.randn(sh, generator=g, device=device), 0).square_(),
                          device)


def config4_device(M: int = 8192, device="cuda") -> LinearProblem:
    """cfg 4 (FFN down-projection, squared-ReLU input) with the tensors drawn on the device."""
    s, N, K = 4000, 5120, 20480
    return LinearProblem(f"cfg4_ffn_down_{M}x{N}x{K}", M, N, K, squared_relu_bf16_device((M, K), s + X_ID, device),
                         normal_bf16_device((N, K), 0.01, s + W_ID, device),
                         normal_bf16_device((M, N), 1e-4, s + DY_ID, device))


def config5_layer_device(layer: int, M: int = 16384, device="cuda") -> LinearProblem:
    """One of the four linears of a transformer block at 16384 tokens, drawn on the device."""
    name, N, K = CONFIG5_LAYERS[layer]
    s = 5000 + 10 * layer
    if name == "ffn_down":
        X = squared_relu_bf16_device((M, K), s + X_ID, device)
    else:
        X = normal_with_outliers_bf16_device((M, K), 0.001, 100.0, s + X_ID, device)
    return LinearProblem(f"cfg5_{name}_{M}x{N}x{K}", M, N, K, X, normal_bf16_device((N, K), 0.02, s + W_ID, device),
                         normal_bf16_device((M, N), 1e-4, s + DY_ID, device), sr_offset=layer)
