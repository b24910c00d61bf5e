"""World-size-2 check of the data-parallel plumbing on CPU (gloo): token sharding, per-rank SR streams and the
FP32 all-reduce of the weight gradient.  The per-rank arithmetic is done by the CPU oracle here; the GPU kernels are
unchanged by data parallelism."""
import os
import socket
import sys
import time

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2509_25149_b200 import dp, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _wgrad(X, dY, rank, mask):
    xq = oracle.quantize(synth.bits(X), colwise=True, rht=True, sign_mask=mask)
    gq = oracle.quantize(synth.bits(dY), colwise=True, rht=True, sign_mask=mask, rounding=oracle.SR, seed=0,
                         sr_offset=dp.rank_sr_offset(rank))
    return oracle.gemm_tn(oracle.dequantize(gq), oracle.dequantize(xq), want_T=False), gq


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        X = synth.normal_bf16((512, 64), 1.0, 1)
        dY = synth.normal_bf16((512, 48), 1e-3, 2)
        b, e = dp.token_shard(512, rank, world)
        dW_local, _ = _wgrad(X[b:e], dY[b:e], rank, synth.DEFAULT_RHT_SIGN_MASK)
        dW = torch.from_numpy(dW_local.astype(np.float32))
        shard = torch.empty((48 // world, 64), dtype=torch.float32)
        dp.reduce_scatter_weight_grad(dW.clone(), shard)
        ref = dW.clone()
        dp.allreduce_weight_grad(ref)
        work = dp.allreduce_weight_grad(dW, async_op=True)  # the overlapped form used by the bench at N > 1
        dp.wait_weight_grad(work)
        assert torch.equal(ref, dW), "asynchronous all-reduce differs from the blocking one"
        b0, e0 = dp.weight_grad_shard(48, rank, world)
        assert torch.equal(shard, dW[b0:e0]), "reduce-scatter shard differs from the rows of the all-reduced dW"
        # the overlapped exchange the bench uses at N > 1: buffers alternate, each step's sum is complete when the
        # buffer comes round again (and after drain)
        ex = dp.OverlappedGradExchange(torch.zeros(6))
        assert len(ex.buffers) == 2
        seen = []
        for step in range(5):
            buf = ex.acquire()
            if step >= 2:
                seen.append(buf.clone())  # the exchange started two steps ago has finished
            buf.fill_(float(step * 10 + rank + 1))
            ex.release(buf)
        ex.drain()
        want = lambda st: float(sum(st * 10 + r + 1 for r in range(world)))
        assert [float(t[0]) for t in seen] == [want(0), want(1), want(2)]
        assert float(ex.buffers[1][0]) == want(3) and float(ex.buffers[0][0]) == want(4)
        # replicated weights quantize to identical bytes on every rank (deterministic RNE)
        W = synth.normal_bf16((48, 64), 0.02, 3)
        wq = torch.from_numpy(oracle.quantize(synth.bits(W), block_rows=16).codes.copy())
        gathered = [torch.empty_like(wq) for _ in range(world)]
        dist.all_gather(gathered, wq)
        assert all(torch.equal(g, wq) for g in gathered)
        if rank == 0:
            np.save(out, dW.numpy())
    finally:
        dist.destroy_process_group()


def test_two_rank_weight_gradient_allreduce(tmp_path):
    out = str(tmp_path / "dw.npy")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = np.load(out)
    X = synth.normal_bf16((512, 64), 1.0, 1)
    dY = synth.normal_bf16((512, 48), 1e-3, 2)
    parts, streams = [], []
    for r in range(2):
        b, e = dp.token_shard(512, r, 2)
        d, gq = _wgrad(X[b:e], dY[b:e], r, synth.DEFAULT_RHT_SIGN_MASK)
        parts.append(d.astype(np.float32))
        streams.append(gq)
    assert np.allclose(got, parts[0] + parts[1], rtol=1e-6, atol=0)
    exact = dY.double().numpy().T @ X.double().numpy()
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.3
    # the two ranks draw from different Philox streams
    assert dp.rank_sr_offset(0) != dp.rank_sr_offset(1)
    assert oracle.sr_draw(0, dp.rank_sr_offset(0), 5) != oracle.sr_draw(0, dp.rank_sr_offset(1), 5) or \
        oracle.sr_draw(0, dp.rank_sr_offset(0), 6) != oracle.sr_draw(0, dp.rank_sr_offset(1), 6)


def test_token_shard_and_offsets():
    assert dp.token_shard(8192, 0, 4) == (0, 2048) and dp.token_shard(8192, 3, 4) == (6144, 8192)
    assert dp.rank_sr_offset(3, 7) == (3 << 32) | 7
    t = torch.ones(4)
    dp.allreduce_weight_grad(t)  # no process group: no-op
    assert dp.allreduce_weight_grad(t, async_op=True) is None
    dp.wait_weight_grad(None)
    assert torch.equal(t, torch.ones(4))
    ex = dp.OverlappedGradExchange(t)  # one buffer, exchange is a no-op
    assert len(ex.buffers) == 1 and ex.acquire() is t
    ex.release(t)
    ex.drain()
    o = torch.empty(4)
    dp.reduce_scatter_weight_grad(t, o)
    assert torch.equal(o, t) and dp.weight_grad_shard(20480, 1, 8) == (2560, 5120)


# ---------------------------------------------------------------------------------------------------------------
# The rank loop of bench.py (barrier, exactly K steps, drain, barrier; time = max over ranks; overlapped exchange of
# the weight gradient) driven by a stub step on two gloo ranks
# ---------------------------------------------------------------------------------------------------------------
def _loop_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    ranks = dp.Ranks("gloo")
    try:
        assert (ranks.world, ranks.rank, ranks.local) == (world, rank, rank) and not ranks.cuda
        ex = dp.OverlappedGradExchange(torch.zeros(4))
        calls = {"n": 0}

        def step():  # stands for fwd + bwd: "Wgrad" writes the buffer, the exchange sums it across ranks
            buf = ex.acquire()
            buf.fill_(float(calls["n"] + 1) * (rank + 1))
            ex.release(buf)
            calls["n"] += 1
            time.sleep(0.002 * (rank + 1))  # rank 1 is the slow one

        t = [0.0]
        start = lambda: t.__setitem__(0, time.perf_counter())
        stop = lambda: (time.perf_counter() - t[0]) * 1e3
        blocks = dp.timed_blocks(ranks, step, ex.drain, steps=5, blocks=3, start=start, stop=stop)
        assert calls["n"] == 15 and len(blocks) == 3
        assert all(b >= 0.002 * world * 1e3 * 0.9 for b in blocks), blocks  # the maximum over ranks: the slow rank's time
        last = ex.buffers[(calls["n"] - 1) % 2]
        assert float(last[0]) == 15.0 * sum(r + 1 for r in range(world))  # drained: the last sum is complete
        assert ranks.max_over_ranks(float(rank)) == float(world - 1)
        torch.save(torch.tensor(blocks), os.path.join(out_dir, f"blocks{rank}.pt"))
    finally:
        ranks.close()


def test_bench_rank_loop_with_a_stub_step(tmp_path):
    mp.spawn(_loop_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    b0, b1 = torch.load(tmp_path / "blocks0.pt"), torch.load(tmp_path / "blocks1.pt")
    assert torch.equal(b0, b1)  # every rank reports the same (maximum) time


def test_spawn_ranks_starts_one_process_per_rank(tmp_path):
    """`bench.py --gpus N` without a launcher re-runs itself through dp.spawn_ranks; here a two-line rank script."""
    script = tmp_path / "rank_script.py"
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script.write_text(
        "import os, sys\n"
        f"sys.path.insert(0, {root!r})\n"
        "from paper_2509_25149_b200 import dp\n"
        "r = dp.Ranks('gloo')\n"
        "r.barrier()\n"
        "open(os.path.join(sys.argv[1], f'rank{r.rank}of{r.world}'), 'w').write(str(r.max_over_ranks(float(r.rank))))\n"
        "r.close()\n")
    assert dp.spawn_ranks(2, str(script), [str(tmp_path)]) == 0
    assert (tmp_path / "rank0of2").read_text() == "1.0" and (tmp_path / "rank1of2").read_text() == "1.0"
