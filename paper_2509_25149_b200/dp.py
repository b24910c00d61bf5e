"""Data-parallel plumbing of the NVFP4 linear layer (one process per GPU, torch.distributed).

The path shards by tokens: every rank quantizes its own X / dY shard (own per-tensor amax, own stochastic-rounding
stream) and runs Fprop, Dgrad, Wgrad locally; the single exchange is the FP32 sum of the weight gradient across
replicas (paper Section 4.1: weight gradients are accumulated in FP32 across data-parallel replicas).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist


def rank_sr_offset(rank: int, layer: int = 0) -> int:
    """Philox counter words 2..3 for a rank: the rank in the high word, the layer index in the low word."""
    assert 0 <= rank < (1 << 31) and 0 <= layer < (1 << 32)
    return (rank << 32) | layer


def token_shard(total_tokens: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of the rank's tokens; shards are multiples of 256 tokens (the linear layer's granularity)."""
    assert total_tokens % (256 * world) == 0, "tokens must split into multiples of 256 per rank"
    per = total_tokens // world
    return rank * per, (rank + 1) * per


def allreduce_weight_grad(dW: torch.Tensor, async_op: bool = False):
    """In-place FP32 sum of dW over all ranks (no-op without an initialised process group).

    async_op=True returns the collective's work handle (None without a process group): the exchange then runs
    beside the next layer's / next step's kernels, and the caller waits on the handle before dW is read or
    overwritten (`wait_weight_grad`)."""
    assert dW.dtype == torch.float32
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        return dist.all_reduce(dW, op=dist.ReduceOp.SUM, async_op=async_op) if async_op else \
            dist.all_reduce(dW, op=dist.ReduceOp.SUM)
    return None


def wait_weight_grad(work) -> None:
    """Blocks the current stream (NCCL) or the caller (gloo) until an asynchronous exchange has finished."""
    if work is not None:
        work.wait()


def weight_grad_shard(n_rows: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of the rows of dW a rank owns when the optimizer state is sharded (rows split evenly)."""
    assert n_rows % world == 0, "output features must split evenly across ranks"
    per = n_rows // world
    return rank * per, (rank + 1) * per


def reduce_scatter_weight_grad(dW: torch.Tensor, out: torch.Tensor) -> None:
    """FP32 sum of dW over all ranks, each rank receiving only its own row shard (`weight_grad_shard`) in `out`:
    the exchange for a sharded optimizer, half the bytes of the all-reduce.  Without a process group `out` is a
    copy of dW."""
    assert dW.dtype == torch.float32 and out.dtype == torch.float32 and dW.is_contiguous() and out.is_contiguous()
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        assert out.numel() * dist.get_world_size() == dW.numel()
        dist.reduce_scatter_tensor(out, dW, op=dist.ReduceOp.SUM)
    else:
        assert out.numel() == dW.numel()
        out.copy_(dW.view_as(out))


class OverlappedGradExchange:
    """Weight-gradient buffers whose exchange runs beside the next step's kernels.

    Each step takes a buffer (`acquire`: waits for the exchange that buffer was last handed to), lets the Wgrad GEMM
    write it, and hands it back (`release`: starts the asynchronous FP32 all-reduce).  With two buffers the exchange
    of step i overlaps the forward and backward kernels of step i + 1; `drain` waits for everything in flight.
    Without a process group (one GPU) there is one buffer and the exchange is a no-op."""

    def __init__(self, like: torch.Tensor, n_buffers: int = 2):
        multi = dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1
        n = max(1, n_buffers) if multi else 1
        self.buffers = [like] + [torch.empty_like(like) for _ in range(n - 1)]
        self.pending = [None] * n
        self.steps = 0

    def acquire(self) -> torch.Tensor:
        i = self.steps % len(self.buffers)
        wait_weight_grad(self.pending[i])
        self.pending[i] = None
        return self.buffers[i]

    def release(self, buf: torch.Tensor) -> None:
        i = self.steps % len(self.buffers)
        assert buf is self.buffers[i], "release the buffer of the current step"
        self.pending[i] = allreduce_weight_grad(buf, async_op=True)
        self.steps += 1

    def drain(self) -> None:
        for i, w in enumerate(self.pending):
            wait_weight_grad(w)
            self.pending[i] = None


# ---------------------------------------------------------------------------------------------
# Rank plumbing of a benchmark / training loop: one process per GPU, started by torch.distributed.run (or by
# `spawn_ranks`, which starts it), the timed region bracketed by a barrier on both sides and timed as the maximum
# over ranks.  Backend "nccl" for GPUs, "gloo" for the CPU tests of the same loop.
# ---------------------------------------------------------------------------------------------
def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, script: str, argv: list[str]) -> int:
    """Re-runs `script argv` as n ranks on this node under torch.distributed.run (rendezvous on 127.0.0.1);
    the ranks' output goes to this process's stdout / stderr.  Returns the launcher's exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(free_port()), script, *argv]
    return subprocess.run(cmd).returncode


class Ranks:
    """World size, rank and local rank from the launcher's environment, and the process group built from them."""

    def __init__(self, backend: str, cuda_device: int | None = None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.cuda = backend == "nccl"
        self.device = torch.device("cuda", self.local if cuda_device is None else cuda_device) if self.cuda else torch.device("cpu")
        if self.world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            if self.cuda:
                dist.init_process_group("nccl", device_id=self.device)
            else:
                dist.init_process_group(backend)

    def barrier(self) -> None:
        if self.world > 1:
            dist.barrier()
        if self.cuda:
            torch.cuda.synchronize()

    def max_over_ranks(self, value: float) -> float:
        if self.world == 1:
            return value
        t = torch.tensor([value], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def close(self) -> None:
        if self.world > 1 and dist.is_initialized():
            dist.destroy_process_group()


def timed_blocks(ranks: Ranks, step, drain, steps: int, blocks: int, start, stop) -> list[float]:
    """`blocks` timed regions of exactly `steps` calls of step() followed by drain(), each bracketed by a barrier on
    both sides; start() / stop() are the caller's timer (stop returns the region's milliseconds).  Returns the
    milliseconds per step of every block, maximum over ranks."""
    out = []
    for _ in range(blocks):
        ranks.barrier()
        start()
        for _ in range(steps):
            step()
        drain()
        ms = stop()
        ranks.barrier()
        out.append(ranks.max_over_ranks(ms / steps))
    return out
