"""Benchmark of the NVFP4 linear-layer hot path on B200.

One step = one pass of the whole path over the FFN up-projection of the 12B-class model
(tokens M = 8192, K = 5120, N = 20480): quantize W (16x16 blocks, both copies), quantize X (row-wise +
rotated column-wise), Fprop, quantize dY (stochastic rounding, row-wise + rotated column-wise), Dgrad, Wgrad.
With --gpus N each rank runs the step on its own 8192-token shard (data parallel, weak scaling) and the FP32
weight gradient is summed across ranks with one NCCL all-reduce.  Under torch.distributed.run the ranks come from the
environment; a plain `python bench.py --gpus N` starts the N ranks itself (re-running this script under
torch.distributed.run, rendezvous on 127.0.0.1).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded slab of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "NVFP4 GEMM TFLOP/s vs FP4 peak; quantize+RHT+SR GB/s vs HBM peak"
M, N, K = 8192, 20480, 5120
WORKLOAD = "cfg3_ffn_up_fwd_bwd_M8192_K5120_N20480"
# DRAM bytes (read + write).  GEMMs: one-pass ncu capture of this workload at full size, cold caches
# (profiles/dram_traffic_cfg3_step.md): the step's two GEMM launches divided by its three GEMMs.  Quantizer: ncu
# captures of the three pass-2 kernels on the reduced --case shapes (profiles/quantize_kernel_dy_x_w.md), 2.80 / 2.73 /
# 2.72 B per element for W / X / dY, scaled to the step's tensors by their element counts (traffic grows in
# proportion), plus the amax passes at the 2 B per element the earlier full-size capture measured for them.
GEMM_DRAM_BYTES_PER_LAUNCH = (547.2e6 + 1092.6e6) / 3  # Fprop launch + merged Dgrad/Wgrad launch, per GEMM
QUANT_DRAM_BYTES_PER_STEP = (N * K) * (2.80 + 2.0) + (M * K) * (2.73 + 2.0) + (M * N) * (2.72 + 2.0)
SLAB = (4096, 2048, 5120)     # tokens, out-features, in-features of the CPU-baseline sample (one run)
SLAB_REF = (512, 1024, 5120)  # per-step sample of the `--impl reference` arm (many steps)


def step_flops(m=M, n=N, k=K) -> float:
    return 3 * 2.0 * m * n * k


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------ clocks ----
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([time.time()] + [t.strip() for t in line.split(",")])

    def median_sm_mhz(self, t0: float, t1: float):
        """Median SM clock of the samples taken between two host times (None if there is none)."""
        v = []
        for r in list(self.rows):
            try:
                if t0 <= r[0] <= t1:
                    v.append(float(r[1]))
            except (ValueError, IndexError):
                continue
        return statistics.median(v) if v else None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx = float(r[2])
                for nme, v in zip(names, r[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(nme)
            except (ValueError, IndexError):
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------ CPU oracle baseline ----
def oracle_slab_step(prob_slices):
    """One fwd+bwd of the slab with the CPU oracle, as it stands.  Returns seconds."""
    import oracle
    from paper_2509_25149_b200 import synth
    X, W, dY, mask = prob_slices
    t0 = time.perf_counter()
    xb, wb, gb = synth.bits(X), synth.bits(W), synth.bits(dY)
    w_row = oracle.quantize(wb, block_rows=16)
    w_col = oracle.quantize(wb, block_rows=16, colwise=True)
    x_row = oracle.quantize(xb)
    x_col = oracle.quantize(xb, colwise=True, rht=True, sign_mask=mask)
    oracle.gemm_tn(oracle.dequantize(x_row), oracle.dequantize(w_row), want_T=False)
    g_row = oracle.quantize(gb, rounding=oracle.SR)
    g_col = oracle.quantize(gb, colwise=True, rht=True, sign_mask=mask, rounding=oracle.SR)
    oracle.gemm_tn(oracle.dequantize(g_row), oracle.dequantize(w_col), want_T=False)
    oracle.gemm_tn(oracle.dequantize(g_col), oracle.dequantize(x_col), want_T=False)
    return time.perf_counter() - t0


def slab_inputs(slab=SLAB):
    from paper_2509_25149_b200 import synth
    ms, ns, ks = slab
    X = synth.normal_with_outliers_bf16((ms, ks), 0.001, 100.0, 3001, 3004)
    W = synth.normal_bf16((ns, ks), 0.02, 3002)
    dY = synth.normal_bf16((ms, ns), 1e-4, 3003)
    return X, W, dY, synth.DEFAULT_RHT_SIGN_MASK


def cpu_baseline(steps=1):
    import oracle
    oracle.build()
    inputs = slab_inputs()
    times = [oracle_slab_step(inputs) for _ in range(steps)]
    ms, ns, ks = SLAB
    t = sum(times) / len(times)
    return {"value": step_flops(ms, ns, ks) / t / 1e12, "unit": "TFLOP/s", "cores": len(os.sched_getaffinity(0)),
            "kind": "oracle",
            "sample": f"fwd+bwd of a {ms}x{ns}x{ks} slab of the workload (tokens 0..{ms - 1}, output features "
                      f"0..{ns - 1}, all {ks} input features): 7 oracle quantize calls + 3 FP64 GEMMs, {t:.2f} s"}, t


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    inputs = slab_inputs(SLAB_REF)
    for _ in range(args.warmup):
        oracle_slab_step(inputs)
    times = [oracle_slab_step(inputs) for _ in range(args.steps)]
    ms, ns, ks = SLAB_REF
    t = sum(times) / len(times)
    val = step_flops(ms, ns, ks) / t / 1e12
    cores = len(os.sched_getaffinity(0))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": f"{ms}x{ns}x{ks} slab per step"},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                             "sample": f"fwd+bwd of a {ms}x{ns}x{ks} slab of the workload per step"},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ CUDA arm ----
def run_cuda(args):
    import torch
    import torch.distributed as dist

    from paper_2509_25149_b200 import binding as B
    from paper_2509_25149_b200 import dp, synth

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    ranks = dp.Ranks("nccl")
    world, rank, local = ranks.world, ranks.rank, ranks.local
    B.lib()
    if args.gemm_tile:
        B.nvfp4_set_gemm_tile_n(args.gemm_tile)

    # inputs: rank r owns its own 8192-token shard (different seeds per rank), W is replicated
    p = synth.config3()
    if rank > 0:
        p.X = synth.normal_with_outliers_bf16((M, K), 0.001, 100.0, 3001 + 100 * rank, 3004 + 100 * rank)
        p.dY = synth.normal_bf16((M, N), 1e-4, 3003 + 100 * rank)
    hX, hW, hdY = p.X.pin_memory(), p.W.pin_memory(), p.dY.pin_memory()
    X, W, dY = hX.cuda(), hW.cuda(), hdY.cuda()
    # --format mxfp4: the same step in the paper's comparison format (extra measurement; the default is NVFP4)
    mx = args.format == "mxfp4"
    fmt = B.FORMAT_MXFP4 if mx else B.FORMAT_NVFP4
    sign_mask = (p.rht_sign_mask | (0xA5C3 << 16)) if mx else p.rht_sign_mask  # 32 sign bits for the 32-point transform
    alloc = lambda r, c: B.alloc_tensor(r, c, format=fmt)
    opts = B.quant_opts(rht_sign_mask=sign_mask, seed=0, sr_offset=dp.rank_sr_offset(rank))
    X_col, W_row, W_col = alloc(K, M), alloc(N, K), alloc(K, N)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((N, K), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")

    # N > 1: the FP32 all-reduce of dW runs beside the next step's kernels (two dW buffers alternate, a buffer is
    # rewritten only after its own exchange has finished); every step's exchange is inside the timed region, the
    # last one is waited for before the closing event
    exchange = dp.OverlappedGradExchange(dW)

    def step():
        buf = exchange.acquire()
        B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)
        B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, buf, False, ws_b)
        exchange.release(buf)  # asynchronous all-reduce; a no-op at N = 1

    drain = exchange.drain
    barrier, max_over_ranks = ranks.barrier, ranks.max_over_ranks

    for _ in range(max(args.warmup, 3)):
        step()
    drain()
    B.nvfp4_device_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # ---- declared pre-load: the same step for >= args.preload seconds, so that the timed blocks start from the clock
    # and power state of a loaded part (the step is power-capped: a region timed right after a pause runs ~10 % fast)
    t_pre = time.perf_counter()
    preload_steps = 0
    while True:
        for _ in range(20):
            step()
        drain()
        torch.cuda.synchronize()
        preload_steps += 20
        if max_over_ranks(time.perf_counter() - t_pre) >= args.preload:
            break
    preload_s = time.perf_counter() - t_pre
    # ---- timed region: args.blocks blocks of EXACTLY args.steps steps, device-resident inputs, each bracketed by a
    # barrier + synchronize on both sides and timed with CUDA events (max over ranks); the median block is reported
    ev = [torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)]
    spans, launch_marks = [], []

    def t_start():
        launch_marks.append(B.nvfp4_launch_count())
        spans.append([time.time(), None])
        ev[0].record()

    def t_stop():
        ev[1].record()
        torch.cuda.synchronize()
        spans[-1][1] = time.time()
        launch_marks[-1] = B.nvfp4_launch_count() - launch_marks[-1]
        return ev[0].elapsed_time(ev[1])

    block_ms = dp.timed_blocks(ranks, step, drain, args.steps, args.blocks, t_start, t_stop)
    ms_step = statistics.median(block_ms)
    launches = launch_marks[block_ms.index(ms_step)] if ms_step in block_ms else launch_marks[0]
    block_mhz = [sampler.median_sm_mhz(a, b) if rank == 0 else None for a, b in spans]
    B.nvfp4_device_status()

    # ---- the same step with the quantized weight reused (micro-batches between optimizer steps): extra figure ----
    def step_cached():
        buf = exchange.acquire()
        B.nvfp4_linear_fwd(X, None, opts, Y, X_col, W_row, W_col, True, ws_f)
        B.nvfp4_linear_bwd(dY, X_col, W_col, K, opts, dX, buf, False, ws_b)
        exchange.release(buf)

    # blocks of 20 steps alternate between the two variants so that both see the same clocks (the step is
    # power-capped: a block timed right after another one inherits its clock state)
    def timed_block(fn, n=20):
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for _ in range(n):
            fn()
        drain()
        b1.record()
        torch.cuda.synchronize()
        return b0.elapsed_time(b1) / n

    barrier()
    alt = {"full": [], "cached": []}
    for _ in range(8):
        alt["full"].append(timed_block(step))
        alt["cached"].append(timed_block(step_cached))
    barrier()
    ms_alt_full = max_over_ranks(sum(alt["full"]) / len(alt["full"]))
    ms_step_cached = max_over_ranks(sum(alt["cached"]) / len(alt["cached"]))
    # ---- per-kernel pass: the same sequence as separate C-ABI calls with events around each ----
    x_row = alloc(M, K)
    g_row, g_col = alloc(M, N), alloc(N, M)
    w_opts = B.quant_opts(block_rows=32 if mx else 16)
    x_opts = B.quant_opts(rht_colwise=True, rht_sign_mask=sign_mask)
    g_opts = B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=sign_mask, seed=0,
                          sr_offset=dp.rank_sr_offset(rank))
    calls = [
        ("quant_W", lambda: B.nvfp4_quantize(W, w_opts, W_row, W_col)),
        ("quant_X", lambda: B.nvfp4_quantize(X, x_opts, x_row, X_col)),
        ("gemm_fprop", lambda: B.nvfp4_gemm(x_row, W_row, Y)),
        ("quant_dY", lambda: B.nvfp4_quantize(dY, g_opts, g_row, g_col)),
        ("gemm_dgrad", lambda: B.nvfp4_gemm(g_row, W_col, dX)),
        ("gemm_wgrad", lambda: B.nvfp4_gemm(g_col, X_col, dW)),
        # the forward call as the step runs it: the amax pass of W rides on the quantize kernel of X and each kernel
        # sets itself up while the one before it drains, which the three separate calls above cannot show
        ("linear_fwd", lambda: B.nvfp4_linear_fwd(X, W, opts, Y, X_col, W_row, W_col, False, ws_f)),
    ]
    per = {name: [] for name, _ in calls}
    t_kern0 = time.time()
    for it in range(min(args.steps, 100) + 2):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
        evs[0].record()
        for i, (_, fn) in enumerate(calls):
            fn()
            evs[i + 1].record()
        torch.cuda.synchronize()
        if it >= 2:
            for i, (name, _) in enumerate(calls):
                per[name].append(evs[i].elapsed_time(evs[i + 1]))
    B.nvfp4_device_status()
    kern_mhz = sampler.median_sm_mhz(t_kern0, time.time()) if rank == 0 else None
    kern_ms = {k: sum(v) / len(v) for k, v in per.items()}

    # Context only (never on the path): the vendor library's block-scaled FP4 GEMM (cuBLASLt through
    # torch._scaled_mm) on the very operand bytes of the three GEMMs, alternating with this repo's kernel in one
    # process.  It shows what a tuned kernel reaches on this part under the same power state.  bf16 outputs for all
    # three (the library call has no fp32-accumulate form here), so the Wgrad pair is timed with a bf16 output too.
    lib_ref = None
    if rank == 0 and not mx and hasattr(torch, "float4_e2m1fn_x2"):
        try:
            f4, f8 = torch.float4_e2m1fn_x2, torch.float8_e4m3fn
            trio = {"gemm_fprop": (x_row, W_row, Y), "gemm_dgrad": (g_row, W_col, dX),
                    "gemm_wgrad": (g_col, X_col, torch.empty((N, K), dtype=torch.bfloat16, device="cuda"))}
            lib_ref = {}
            for name, (a, b, d) in trio.items():
                a4, b4t = a.codes.view(f4), b.codes.view(f4).t()
                sa, sb = a.scales.view(f8), b.scales.view(f8)
                fns = {"this_repo_ms": lambda: B.nvfp4_gemm(a, b, d),
                       "library_ms": lambda: torch._scaled_mm(a4, b4t, sa, sb, out_dtype=torch.bfloat16)}
                acc = {k: [] for k in fns}
                for _ in range(4):
                    for k, fn in fns.items():
                        acc[k].append(timed_block(fn, 10))
                lib_ref[name] = {k: round(statistics.median(v), 4) for k, v in acc.items()}
        except Exception as exc:  # the call is context, not a dependency
            lib_ref = {"unavailable": repr(exc)[:160]}

    # the same layer kept in BF16 (Section 4.1 leaves a share of the layers in higher precision): context for the
    # FP4 step, no exchange, timed in the same alternation
    def step_bf16():
        B.nvfp4_linear_bf16_fwd(X, W, Y)
        B.nvfp4_linear_bf16_bwd(dY, X, W, K, dX, dW)

    # a second alternation for the BF16 layer: its dense BF16 GEMMs pull the clocks further down than the FP4 step
    # does, so the FP4 blocks beside it run slower than in the loop above; the ratio is taken inside this loop
    for _ in range(2):
        step_bf16()
    alt2 = {"full": [], "bf16": []}
    for _ in range(4):
        alt2["full"].append(timed_block(step, 10))
        alt2["bf16"].append(timed_block(step_bf16, 10))
    barrier()
    ms_full_beside_bf16 = max_over_ranks(sum(alt2["full"]) / len(alt2["full"]))
    ms_step_bf16 = max_over_ranks(sum(alt2["bf16"]) / len(alt2["bf16"]))

    # ---- end to end: host buffers, copies inside the timed region --------------------------------
    hY = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    hdX = torch.empty((M, K), dtype=torch.bfloat16).pin_memory()
    hdW = torch.empty((N, K), dtype=torch.float32).pin_memory()

    # Copies and kernels of neighbouring steps overlap: inputs and outputs are double-buffered on the device, the
    # host->device copies of step i+1 and the device->host copies of step i-1 run on their own streams beside the
    # kernels of step i.  Every step still moves all of its inputs and all of its results.
    drain()
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ins = [(X, W, dY), (torch.empty_like(X), torch.empty_like(W), torch.empty_like(dY))]
    outs = [(Y, dX, dW), (torch.empty_like(Y), torch.empty_like(dX), torch.empty_like(dW))]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        b = i & 1
        Xb, Wb, dYb = ins[b]
        Yb, dXb, dWb = outs[b]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[b])  # step i-2 has consumed this input buffer
            Xb.copy_(hX, non_blocking=True)
            Wb.copy_(hW, non_blocking=True)
            dYb.copy_(hdY, non_blocking=True)
            ev_in[b].record(s_in)
        cur.wait_event(ev_in[b])
        cur.wait_event(ev_out[b])        # the results of step i-2 have left this output buffer
        B.nvfp4_linear_fwd(Xb, Wb, opts, Yb, X_col, W_row, W_col, False, ws_f)
        B.nvfp4_linear_bwd(dYb, X_col, W_col, K, opts, dXb, dWb, False, ws_b)
        dp.allreduce_weight_grad(dWb)
        ev_comp[b].record(cur)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            hY.copy_(Yb, non_blocking=True)
            hdX.copy_(dXb, non_blocking=True)
            hdW.copy_(dWb, non_blocking=True)
            ev_out[b].record(s_out)

    e2e_steps = max(4, min(args.steps, 10))
    e2e_step(0)
    e2e_step(1)
    cur.wait_stream(s_in)
    cur.wait_stream(s_out)
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    cur.wait_stream(s_in)
    cur.wait_stream(s_out)
    t1.record()
    barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1) / e2e_steps)
    h2d = sum(t.numel() * t.element_size() for t in (hX, hW, hdY))
    d2h = sum(t.numel() * t.element_size() for t in (hY, hdX, hdW))

    if rank == 0:
        clocks = sampler.stop()
        # the clock record of the timed blocks themselves (the key the timing rules ask for), the whole run beside it
        timed_mhz = [m for m in block_mhz if m is not None]
        clocks["sm_mhz_whole_run"] = clocks["sm_mhz"]
        if timed_mhz:
            clocks["sm_mhz"] = statistics.median(timed_mhz)
        peaks = measured_peaks()
        flops = step_flops()
        gemm_ms = (kern_ms["gemm_fprop"] + kern_ms["gemm_dgrad"] + kern_ms["gemm_wgrad"]) / 3
        gemm_tflops = 2.0 * M * N * K / (gemm_ms * 1e-3) / 1e12
        # FP4 : BF16 dense = 4 : 1 (nominal ratio).  The denominator is the BURST bf16 figure: the GEMMs are timed one
        # launch at a time between cooler quantizer kernels, not in a seconds-long GEMM-only loop
        fp4_peak = 4.0 * peaks["bf16_tflops"]
        per_gemm = {k: 2.0 * M * N * K / (kern_ms[k] * 1e-3) / 1e12 for k in ("gemm_fprop", "gemm_dgrad", "gemm_wgrad")}
        # tensor-pipe occupancy at the sampled clock: 16384 dense FP4 MAC / clock / SM x 148 SMs (the 9 PFLOP/s of the
        # datasheet correspond to 1.86 GHz at that rate; a derived figure, NVIDIA does not publish the per-SM rate)
        mac_clk_sm, n_sm = 16384, 148
        pipe = (lambda tf: tf * 1e12 / (kern_mhz * 1e6 * n_sm * mac_clk_sm * 2)) if kern_mhz else (lambda tf: None)
        # quantizer: algorithmic bytes = two reads of the bf16 tensor + both copies (codes + scales)
        q_elems = M * K + N * K + M * N
        # (MXFP4 has no tensor-level scale, hence one read, and one scale byte per 32 elements)
        bpe = (2 + 2 * (0.5 + 1.0 / 32)) if mx else (2 + 2 + 2 * (0.5 + 1.0 / 16))  # algorithmic bytes per element
        q_bytes = q_elems * bpe
        # quantizer time of the step: the forward call minus its GEMM timed alone (the composed call fuses W's amax
        # pass into X's quantize kernel), plus the dY quantize call; the separate calls stay in per_tensor
        q_fwd_ms = kern_ms.pop("linear_fwd") - kern_ms["gemm_fprop"]
        q_ms_separate = kern_ms["quant_W"] + kern_ms["quant_X"] + kern_ms["quant_dY"]
        q_ms = (q_fwd_ms if not mx else kern_ms["quant_W"] + kern_ms["quant_X"]) + kern_ms["quant_dY"]
        q_gbs = q_bytes / (q_ms * 1e-3) / 1e9
        cpu, _ = cpu_baseline(1) if not (args.no_cpu_baseline or mx) else (None, 0)
        line = {
            "metric": METRIC, "value": world * flops / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
            # the timed region: args.blocks blocks of `steps` steps after a declared pre-load; ms_per_step is the median
            # block; cycles_per_step = ms x median SM MHz of that block's samples (a clock-free figure)
            "timing": {"preload_s": round(preload_s, 3), "preload_steps": preload_steps, "blocks": args.blocks,
                       "block_ms_per_step": [round(b, 4) for b in block_ms],
                       "block_sm_mhz": block_mhz,
                       "mcycles_per_step": [round(b * m / 1e3, 1) if m else None for b, m in zip(block_ms, block_mhz)]},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4_e2m1",
            "data": "synthetic",
            "config": {"workload": WORKLOAD + ("_mxfp4" if mx else ""), "tokens_per_gpu": M, "in_features": K,
                       "out_features": N,
                       "parallelism": f"dp{world}", "l2": "inputs (629 MB bf16 per step) exceed the 126 MB L2",
                       "step": "quantize W (2D), quantize X, Fprop, quantize dY (SR), Dgrad, Wgrad"
                               + (", FP32 all-reduce of dW" if world > 1 else "")},
            # extra: the step with the quantized weight reused (no quantize W), and the full step again, timed in
            # alternating blocks of 20 steps
            "ms_per_step_w_cached": ms_step_cached, "ms_per_step_alternating": ms_alt_full,
            # extra: the same layer through the BF16 kernels (no quantization), same alternation
            "bf16_layer": {"ms_per_step": ms_step_bf16, "tflops": flops / (ms_step_bf16 * 1e-3) / 1e12,
                           "fp4_ms_per_step_beside_it": ms_full_beside_bf16,
                           "fp4_step_speedup": ms_step_bf16 / ms_full_beside_bf16},
            "gemm_tflops": gemm_tflops, "quant_gbs": q_gbs,
            "kernel_ms": {k: round(v, 4) for k, v in kern_ms.items()},
            "roofline": {"bound": "tensor", "kernel": "gemm_pair_kernel / gemm_wide_kernel (mean of Fprop, Dgrad, Wgrad)",
                         "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
                         "frac": gemm_tflops / fp4_peak, "traffic": None if mx else GEMM_DRAM_BYTES_PER_LAUNCH,
                         "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum, full-size one-pass "
                                           "capture, mean of the three GEMMs (profiles/dram_traffic_cfg3_step.md)",
                         "peak_source": f"4 x {peaks['source']} burst bf16 cuBLAS ({peaks['bf16_tflops']} TFLOP/s)",
                         "frac_of_sustained": gemm_tflops / (4.0 * peaks["bf16_tflops_sustained"]),
                         "frac_of_datasheet_9pf": gemm_tflops / 9000.0,
                         "per_gemm": {k: {"tflops": round(v, 1), "frac": v / fp4_peak, "frac_of_datasheet_9pf": v / 9000.0,
                                          "tensor_pipe_frac": pipe(v)} for k, v in per_gemm.items()},
                         "tensor_pipe_frac": pipe(gemm_tflops), "tensor_pipe_sm_mhz": kern_mhz,
                         "tensor_pipe_rate": "16384 FP4 MAC / clock / SM x 148 SMs (derived from the 9 PFLOP/s datasheet figure)",
                         "library_fp4_gemm_context": lib_ref},
            "roofline_quant": {"bound": "hbm", "kernel": "amax kernels + quantize_kernel (W, X, dY)",
                               "achieved": q_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": q_gbs / peaks["hbm_gbs"], "traffic": None if mx else QUANT_DRAM_BYTES_PER_STEP,
                               "algorithmic_bytes": q_bytes,
                               "peak_source": f"{peaks['source']} copy bandwidth",
                               "frac_of_datasheet_8tbs": q_gbs / 8000.0,
                               "time_ms": {"forward_call_minus_fprop": round(q_fwd_ms, 4),
                                           "quant_dY": round(kern_ms["quant_dY"], 4),
                                           "three_separate_calls": round(q_ms_separate, 4)},
                               "frac_three_separate_calls": q_bytes / (q_ms_separate * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "per_tensor": {k: {"gbs": round(e * bpe / (kern_ms[k] * 1e-3) / 1e9, 1),
                                                  "frac": e * bpe / (kern_ms[k] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                                              for k, e in (("quant_W", N * K), ("quant_X", M * K), ("quant_dY", M * N))}},
            "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                    "overlap": "copies of neighbouring steps overlap the kernels (double-buffered)"},
            "gpu_launches": launches, "clocks": clocks, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    ranks.close()


# ------------------------------------------------- single-kernel cases (profiling) ----
CASES = {
    # name: (kind, rows/M, cols/N, K)
    "gemm_fprop": ("gemm", 4096, 5120, 5120),      # bf16 output, K = 5120
    "gemm_wgrad": ("gemm32", 5120, 5120, 4096),    # fp32 output
    "quant_x": ("qx", 16384, 5120, 0),             # RNE, row-wise + rotated column-wise (168 MB > L2)
    "quant_dy": ("qdy", 4096, 20480, 0),           # SR, row-wise + rotated column-wise (168 MB > L2)
    "quant_w": ("qw", 20480, 5120, 0),             # 16x16 blocks, both copies (210 MB > L2)
    "quant_dy_mx": ("qdy_mx", 4096, 20480, 0),      # MXFP4: SR, row-wise + rotated column-wise, one pass
    "quant_w_mx": ("qw_mx", 20480, 5120, 0),        # MXFP4: 32x32 blocks, both copies
    "gemm_fprop_mx": ("gemm_mx", 4096, 5120, 5120), # MXFP4 operands, bf16 output
    "quant_w_f32": ("qw_f32", 20480, 5120, 0),      # 16x16 blocks, both copies, from a binary32 source (419 MB)
    "step": ("step", 8192, 20480, 5120),           # the whole cfg 3 fwd + bwd step, full size: ONE-PASS captures only
    "fwd_half": ("fwd", 8192, 10240, 5120),         # forward call, half the output features (X 84 MB, W 105 MB): the
                                                    # quantize kernel of X that carries the amax pass of W
    "gemm_bf16_fprop": ("bf16", 4096, 5120, 5120),  # BF16 layer (Section 4.1): Y = X W^T, both operands K-major
    "gemm_bf16_wgrad": ("bf16_wgrad", 5120, 5120, 4096),  # dW = dY^T X, both operands read transposed, fp32 output
    "step_bf16": ("step_bf16", 8192, 20480, 5120),  # the cfg 3 layer kept in BF16, fwd + bwd, full size
    "quant_dy_rht4": ("qdy_rht4", 4096, 20480, 0),    # Appendix E.4.2: 4 x 4 transform
    "quant_dy_rht128": ("qdy_rht128", 4096, 20480, 0),  # Appendix E.4.2: 128 x 128 transform
    "quant_x_rowscale": ("q_rows", 16384, 5120, 0),  # App. B.1 closing remark: one pass, global scale per row, RNE
    "quant_dy_rowscale": ("q_rows_sr", 4096, 20480, 0),  # the same with stochastic rounding on gradient-shaped rows
    "quant_error": ("qerr", 4096, 20480, 0),        # Appendix E.2: decode-and-compare reduction (2.5625 B / element)
    # what bounds a 256-deep k-block of the CTA-pair GEMM: SM cycles and nanoseconds per k-block, measured inside the
    # kernel, for the full loop and with parts switched off, on all 74 SM pairs and on 37 (balanced shape: 6 tiles of
    # 80 k-blocks per pair)
    "gemm_cycles": ("gemm_cycles", 256 * 74, 1536, 20480),
}


def run_case(args):
    """Runs ONE kernel family on a reduced shape: the small, self-terminating target for ncu captures."""
    import torch

    from paper_2509_25149_b200 import binding as B
    from paper_2509_25149_b200 import synth

    kind, r, c, k = CASES[args.case]
    torch.cuda.set_device(0)
    if args.gemm_tile:
        B.nvfp4_set_gemm_tile_n(args.gemm_tile)
    g = torch.Generator(device="cuda").manual_seed(1)
    mask = synth.DEFAULT_RHT_SIGN_MASK
    if kind == "gemm_cycles":
        return run_gemm_cycles(args, r, c, k)
    if kind == "step":
        X = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        W = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        dY = (torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32) * 1e-4).to(torch.bfloat16)
        Y = torch.empty((r, c), dtype=torch.bfloat16, device="cuda")
        dX = torch.empty((r, k), dtype=torch.bfloat16, device="cuda")
        dW = torch.empty((c, k), dtype=torch.float32, device="cuda")
        X_col, W_row, W_col = B.alloc_tensor(k, r), B.alloc_tensor(c, k), B.alloc_tensor(k, c)
        ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(r, k), dtype=torch.uint8, device="cuda")
        ws_b = torch.empty(B.nvfp4_linear_bwd_workspace_bytes(r, c), dtype=torch.uint8, device="cuda")
        o = B.quant_opts(rht_sign_mask=mask, seed=0, sr_offset=0)

        def fn():
            B.nvfp4_linear_fwd(X, W, o, Y, X_col, W_row, W_col, False, ws_f)
            B.nvfp4_linear_bwd(dY, X_col, W_col, k, o, dX, dW, False, ws_b)
        work, unit = 3 * 2.0 * r * c * k / 1e12, "TFLOP/s"
    elif kind == "fwd":
        X = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        W = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        Y = torch.empty((r, c), dtype=torch.bfloat16, device="cuda")
        X_col, W_row, W_col = B.alloc_tensor(k, r), B.alloc_tensor(c, k), B.alloc_tensor(k, c)
        ws_f = torch.empty(B.nvfp4_linear_fwd_workspace_bytes(r, k), dtype=torch.uint8, device="cuda")
        o = B.quant_opts(rht_sign_mask=mask)
        fn = lambda: B.nvfp4_linear_fwd(X, W, o, Y, X_col, W_row, W_col, False, ws_f)
        work, unit = 2.0 * r * c * k / 1e12, "TFLOP/s"
    elif kind == "step_bf16":
        X = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        W = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        dY = (torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32) * 1e-4).to(torch.bfloat16)
        Y = torch.empty((r, c), dtype=torch.bfloat16, device="cuda")
        dX = torch.empty((r, k), dtype=torch.bfloat16, device="cuda")
        dW = torch.empty((c, k), dtype=torch.float32, device="cuda")

        def fn():
            B.nvfp4_linear_bf16_fwd(X, W, Y)
            B.nvfp4_linear_bf16_bwd(dY, X, W, k, dX, dW)
        work, unit = 3 * 2.0 * r * c * k / 1e12, "TFLOP/s"
    elif kind in ("bf16", "bf16_wgrad"):
        if kind == "bf16":
            a = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            b = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
            D = torch.empty((r, c), dtype=torch.bfloat16, device="cuda")
            fn = lambda: B.nvfp4_gemm_bf16(a, b, D)
        else:  # operands stored [tokens][features]: the contraction runs down their rows
            a = torch.randn((k, r), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            b = torch.randn((k, c), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            D = torch.empty((r, c), dtype=torch.float32, device="cuda")
            fn = lambda: B.nvfp4_gemm_bf16(a, b, D, B.MN_MAJOR, B.MN_MAJOR)
        work, unit = 2.0 * r * c * k / 1e12, "TFLOP/s"
    elif kind in ("q_rows", "q_rows_sr"):
        x = torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        row = B.alloc_tensor(r, c, format=B.FORMAT_NVFP4_ROWSCALE)
        o = B.quant_opts(rounding=B.ROUND_STOCHASTIC if kind == "q_rows_sr" else B.ROUND_NEAREST_EVEN, seed=1)
        fn = lambda: B.nvfp4_quantize(x, o, row, None)
        work, unit = r * c * 2.5625 / 1e9, "GB/s"
    elif kind == "qerr":
        x = torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        q = B.alloc_tensor(r, c)
        B.nvfp4_quantize(x, B.quant_opts(), q, None)
        out = torch.empty(2, dtype=torch.float64, device="cuda")
        fn = lambda: B.nvfp4_quant_error(x, q, out)
        work, unit = r * c * 2.5625 / 1e9, "GB/s"
    elif kind in ("qdy_rht4", "qdy_rht128"):
        x = (torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32) * 1e-4).to(torch.bfloat16)
        row, col = B.alloc_tensor(r, c), B.alloc_tensor(c, r)
        o = B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_dim=4 if kind == "qdy_rht4" else 128,
                         rht_sign_mask=0x5A5A73E51234ABCD0F0F3C3C999973E5)
        fn = lambda: B.nvfp4_quantize(x, o, row, col)
        work, unit = r * c * 5.125 / 1e9, "GB/s"
    elif kind == "gemm_mx":
        a_src = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        b_src = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        A, Bq = B.alloc_tensor(r, k, format=B.FORMAT_MXFP4), B.alloc_tensor(c, k, format=B.FORMAT_MXFP4)
        B.nvfp4_quantize(a_src, B.quant_opts(), A, None)
        B.nvfp4_quantize(b_src, B.quant_opts(block_rows=32), Bq, None)
        D = torch.empty((r, c), dtype=torch.bfloat16, device="cuda")
        fn = lambda: B.nvfp4_gemm(A, Bq, D)
        work, unit = 2.0 * r * c * k / 1e12, "TFLOP/s"
    elif kind in ("qdy_mx", "qw_mx"):
        x = torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32)
        x = (x * (1e-4 if kind == "qdy_mx" else 0.02)).to(torch.bfloat16)
        row, col = B.alloc_tensor(r, c, format=B.FORMAT_MXFP4), B.alloc_tensor(c, r, format=B.FORMAT_MXFP4)
        o = (B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=0xA5C373E5)
             if kind == "qdy_mx" else B.quant_opts(block_rows=32))
        fn = lambda: B.nvfp4_quantize(x, o, row, col)
        work, unit = r * c * 3.0625 / 1e9, "GB/s"
    elif kind == "qw_f32":
        x = torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32) * 0.02
        row, col = B.alloc_tensor(r, c), B.alloc_tensor(c, r)
        o = B.quant_opts(block_rows=16)
        fn = lambda: B.nvfp4_quantize(x, o, row, col)
        work, unit = r * c * (4 + 4 + 1.125) / 1e9, "GB/s"
    elif kind in ("gemm", "gemm32"):
        a_src = torch.randn((r, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        b_src = (torch.randn((c, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        A, Bq = B.alloc_tensor(r, k), B.alloc_tensor(c, k)
        B.nvfp4_quantize(a_src, B.quant_opts(), A, None)
        B.nvfp4_quantize(b_src, B.quant_opts(block_rows=16), Bq, None)
        D = torch.empty((r, c), dtype=torch.float32 if kind == "gemm32" else torch.bfloat16, device="cuda")
        fn = lambda: B.nvfp4_gemm(A, Bq, D)
        work, unit = 2.0 * r * c * k / 1e12, "TFLOP/s"
    else:
        x = torch.randn((r, c), generator=g, device="cuda", dtype=torch.float32)
        x = (x * (1e-4 if kind == "qdy" else 0.02 if kind == "qw" else 1.0)).to(torch.bfloat16)
        row, col = B.alloc_tensor(r, c), B.alloc_tensor(c, r)
        o = {"qx": B.quant_opts(rht_colwise=True, rht_sign_mask=mask),
             "qdy": B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True, rht_sign_mask=mask),
             "qw": B.quant_opts(block_rows=16)}[kind]
        fn = lambda: B.nvfp4_quantize(x, o, row, col)
        work, unit = r * c * 5.125 / 1e9, "GB/s"
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    B.nvfp4_device_status()
    ms = e0.elapsed_time(e1) / args.steps
    print(json.dumps({"case": args.case, "shape": [r, c, k], "ms": ms, "value": work / (ms * 1e-3), "unit": unit}))


def run_gemm_cycles(args, m, n, k):
    """Table of SM cycles / nanoseconds / effective SM clock per 256-deep k-block of the CTA-pair GEMM (256 x 256
    tiles), read from the kernel's own cycle and nanosecond counters: everything on, MMAs only, loads only, scale path
    off, each on all SM pairs and on half of them.  The variants alternate inside one process (`--steps` launches per
    turn, 4 turns) so that all see the same box and power state."""
    import torch

    from paper_2509_25149_b200 import binding as B

    g = torch.Generator(device="cuda").manual_seed(1)
    a_src = torch.randn((m, k), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    b_src = (torch.randn((n, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
    A, Bq = B.alloc_tensor(m, k), B.alloc_tensor(n, k)
    B.nvfp4_quantize(a_src, B.quant_opts(), A, None)
    B.nvfp4_quantize(b_src, B.quant_opts(block_rows=16), Bq, None)
    del a_src, b_src
    D = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
    B.nvfp4_set_gemm_tile_n(512)
    n_pairs = torch.cuda.get_device_properties(0).multi_processor_count // 2
    probe = torch.zeros(8 * n_pairs, dtype=torch.int64, device="cuda")
    variants = [("all on", 0), ("no MMAs (loads + scale path)", 1), ("no operand loads (MMAs + scale path)", 2),
                ("no scale path (loads + MMAs)", 4), ("MMAs only", 6),
                ("scale atoms through tcgen05.cp issued by the MMA issuer", 32),
                ("the same, no MMAs", 33)]
    rows = {}
    for turn in range(4):
        for pairs in (n_pairs, n_pairs // 2):
            for name, mode in variants:
                B.nvfp4_set_gemm_experiment(mode, pairs, probe)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                for _ in range(3):
                    B.nvfp4_gemm(A, Bq, D)
                e0.record()
                for _ in range(args.steps):
                    B.nvfp4_gemm(A, Bq, D)
                e1.record()
                torch.cuda.synchronize()
                p = probe.view(-1, 8)[:pairs].cpu().double()  # the last launch's counters
                cyc, ns, kb, tiles, wait = p[:, 0], p[:, 1], p[:, 2], p[:, 3], p[:, 4]
                rows.setdefault((name, pairs), []).append(
                    (float((cyc / kb).median()), float((ns / kb).median()), float((cyc / ns).median()) * 1e3,
                     e0.elapsed_time(e1) / args.steps, float((wait / tiles).median())))
    B.nvfp4_set_gemm_experiment(0, 0, None)
    B.nvfp4_set_gemm_tile_n(0)
    B.nvfp4_device_status()
    table = []
    for (name, pairs), v in rows.items():
        t = torch.tensor(v).median(dim=0).values.tolist()
        table.append({"variant": name, "pairs": pairs, "cycles_per_kblock": round(t[0], 1), "ns_per_kblock": round(t[1], 1),
                      "sm_mhz": round(t[2], 0), "launch_ms": round(t[3], 4),
                      "handover_wait_cycles_per_tile": round(t[4], 0)})
    print(json.dumps({"case": "gemm_cycles", "shape": [m, n, k], "k_blocks_per_pair": (m // 256) * (n // 256) * (k // 256) // n_pairs,
                      "mma_cycles_per_kblock_at_16384_mac_per_clk_sm": 4 * 256 * 256 * 64 / (2 * 16384),
                      "launches_per_turn": args.steps, "turns": 4, "table": table}))


# ------------------------------------------- other 12B-class configs (extra measurements) ----
def run_config(args):
    """Times fwd + bwd of every linear layer of cfg 4 (FFN down) or cfg 5 (all four linears of a block, 16384
    tokens): per-kernel CUDA-event times and the whole sequence.  Inputs are drawn on the device with the shapes
    and distributions of the config (timing only; parity for these shapes is covered by the tests)."""
    import torch

    from paper_2509_25149_b200 import binding as B
    from paper_2509_25149_b200 import synth

    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(1000 * args.config)
    layers = {4: [("ffn_down", 8192, 5120, 20480, True)],
              5: [("qkv", 16384, 7168, 5120, False), ("out_proj", 16384, 5120, 5120, False),
                  ("ffn_up", 16384, 20480, 5120, False), ("ffn_down", 16384, 5120, 20480, True)]}[args.config]
    mask = synth.DEFAULT_RHT_SIGN_MASK
    built = []
    for li, (name, m, n, k, relu2) in enumerate(layers):
        x = torch.randn((m, k), generator=gen, device="cuda", dtype=torch.float32)
        if relu2:
            x = torch.clamp_min(x, 0).square_()
        else:
            x = torch.where(torch.rand((m, k), generator=gen, device="cuda") < 0.001, x * 100.0, x)
        X = x.to(torch.bfloat16)
        del x
        W = (torch.randn((n, k), generator=gen, device="cuda", dtype=torch.float32) * (0.01 if args.config == 4 else 0.02)).to(torch.bfloat16)
        dY = (torch.randn((m, n), generator=gen, device="cuda", dtype=torch.float32) * 1e-4).to(torch.bfloat16)
        bufs = dict(X=X, W=W, dY=dY, x_row=B.alloc_tensor(m, k), X_col=B.alloc_tensor(k, m), W_row=B.alloc_tensor(n, k),
                    W_col=B.alloc_tensor(k, n), g_row=B.alloc_tensor(m, n), g_col=B.alloc_tensor(n, m),
                    Y=torch.empty((m, n), dtype=torch.bfloat16, device="cuda"),
                    dX=torch.empty((m, k), dtype=torch.bfloat16, device="cuda"),
                    dW=torch.empty((n, k), dtype=torch.float32, device="cuda"),
                    ws_f=torch.empty(B.nvfp4_linear_fwd_workspace_bytes(m, k), dtype=torch.uint8, device="cuda"),
                    ws_b=torch.empty(B.nvfp4_linear_bwd_workspace_bytes(m, n), dtype=torch.uint8, device="cuda"),
                    opts=B.quant_opts(rht_sign_mask=mask, seed=0, sr_offset=li))
        built.append((name, m, n, k, bufs))

    def step():
        for name, m, n, k, b in built:
            B.nvfp4_linear_fwd(b["X"], b["W"], b["opts"], b["Y"], b["X_col"], b["W_row"], b["W_col"], False, b["ws_f"])
        for name, m, n, k, b in reversed(built):
            B.nvfp4_linear_bwd(b["dY"], b["X_col"], b["W_col"], k, b["opts"], b["dX"], b["dW"], False, b["ws_b"])

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    B.nvfp4_device_status()
    ms_step = e0.elapsed_time(e1) / args.steps

    out_layers = {}
    tot_flops = tot_qbytes = tot_gemm_ms = tot_q_ms = 0.0
    for name, m, n, k, b in built:
        calls = [
            ("quant_W", lambda: B.nvfp4_quantize(b["W"], B.quant_opts(block_rows=16), b["W_row"], b["W_col"])),
            ("quant_X", lambda: B.nvfp4_quantize(b["X"], B.quant_opts(rht_colwise=True, rht_sign_mask=mask), b["x_row"], b["X_col"])),
            ("gemm_fprop", lambda: B.nvfp4_gemm(b["x_row"], b["W_row"], b["Y"])),
            ("quant_dY", lambda: B.nvfp4_quantize(b["dY"], B.quant_opts(rounding=B.ROUND_STOCHASTIC, rht_colwise=True,
                                                                          rht_sign_mask=mask), b["g_row"], b["g_col"])),
            ("gemm_dgrad", lambda: B.nvfp4_gemm(b["g_row"], b["W_col"], b["dX"])),
            ("gemm_wgrad", lambda: B.nvfp4_gemm(b["g_col"], b["X_col"], b["dW"])),
        ]
        per = {c[0]: [] for c in calls}
        for it in range(12):
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
            evs[0].record()
            for i, (_, fn) in enumerate(calls):
                fn()
                evs[i + 1].record()
            torch.cuda.synchronize()
            if it >= 2:
                for i, (cn, _) in enumerate(calls):
                    per[cn].append(evs[i].elapsed_time(evs[i + 1]))
        km = {c: sum(v) / len(v) for c, v in per.items()}
        g_ms = km["gemm_fprop"] + km["gemm_dgrad"] + km["gemm_wgrad"]
        q_ms = km["quant_W"] + km["quant_X"] + km["quant_dY"]
        q_bytes = (m * k + n * k + m * n) * 5.125
        out_layers[name] = {"M": m, "N": n, "K": k, "kernel_ms": {c: round(v, 4) for c, v in km.items()},
                            "gemm_tflops": round(3 * 2.0 * m * n * k / (g_ms * 1e-3) / 1e12, 1),
                            "quant_gbs": round(q_bytes / (q_ms * 1e-3) / 1e9, 1)}
        tot_flops += 3 * 2.0 * m * n * k
        tot_qbytes += q_bytes
        tot_gemm_ms += g_ms
        tot_q_ms += q_ms
    print(json.dumps({"config": args.config, "ms_per_step": ms_step, "value": tot_flops / (ms_step * 1e-3) / 1e12,
                      "unit": "TFLOP/s", "gemm_tflops": tot_flops / (tot_gemm_ms * 1e-3) / 1e12,
                      "quant_gbs": tot_qbytes / (tot_q_ms * 1e-3) / 1e9, "layers": out_layers, "steps": args.steps,
                      "data": "synthetic (device generator)"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3, choices=[3, 4, 5],
                    help="3 = the benchmark workload (default); 4 / 5 = extra measurements of the other 12B-class configs")
    ap.add_argument("--case", default=None, choices=sorted(CASES), help="run one kernel on a reduced shape")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--blocks", type=int, default=5, help="timed blocks of --steps steps; the median block is reported")
    ap.add_argument("--preload", type=float, default=1.0, help="seconds of the same step run before the timed blocks")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm-tile", type=int, default=0, choices=[0, 128, 256, 512, 768],
                    help="force a GEMM tile configuration (0: the library's choice); for experiments")
    ap.add_argument("--format", default="nvfp4", choices=["nvfp4", "mxfp4"],
                    help="mxfp4: run the step in the paper's comparison format (extra measurement)")
    args = ap.parse_args()
    if args.case:
        run_case(args)
    elif args.config != 3:
        run_config(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain `python bench.py --gpus N`: start the N ranks (one per GPU) ourselves
        from paper_2509_25149_b200 import dp
        sys.exit(dp.spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
