#!/usr/bin/env python
"""Benchmark of the block-structured-pruning hot path on B200.

One *step* = one pass of the whole path over one batch of synthetic input, for each of the four
linears of a BERT-base encoder layer at 4096 tokens (16-row blocks, 3.0x compression):
    norms, gamma, penalty  ->  Algorithm 1 keep flags + packed storage  ->  execution layout
    (bsp_prepare_batched: one call for the four matrices)  ->  bsp_linear_planned (tcgen05 GEMM + bias [+ GELU]),
with the layer's outputs chained (attention-output reads the V third of QKV's output, FFN-up
reads attention-output's result through GELU, FFN-down reads FFN-up's).

    python bench.py --gpus N --steps K --warmup W            # the CUDA path
    python bench.py --impl reference ...                     # the CPU oracle, timed as it stands

The metric is TFLOP/s counted on non-zero multiply-adds: 2 * tokens * kept weights per step.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "block-sparse linear TFLOP/s (nonzero) & % bf16 tensor peak, BERT-base shapes"
UNIT = "TFLOP/s"
EPS = 1e-3
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_FLUSH_BYTES = 256 << 20      # larger than the 126 MB L2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload():
    return si.bert_base_layer(tokens=4096, rate=3.0, block=16)


# ------------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
        0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.period = [], set(), period_s
        self.max_mhz, self._stop, self._thread, self._h, self._nv = None, threading.Event(), None, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            import torch
            uuid = torch.cuda.get_device_properties(device_index).uuid
            self._h = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if str(uuid) in u:
                    self._h = h
            if self._h is None:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
class LayerOnDevice:
    """Device buffers and the per-step call sequence for one rank's batch."""

    def __init__(self, wl, seed, rank, device):
        import torch
        import paper_2009_08065_b200 as bsp
        self.torch, self.bsp, self.wl, self.device = torch, bsp, wl, device
        # The step's inputs (X, the four W, the four biases) live in ONE device buffer and one pinned host
        # buffer, each tensor a 256-byte-aligned view: the end-to-end leg uploads them with a single copy.
        x = si.make_activations(rank_seed(seed, rank), "layer_in", wl.tokens, wl.linears[0].k_in)
        parts = [("x", x.view(np.int16))]
        for spec in wl.linears:
            wp, _ = si.make_pruned_weight(seed, spec)          # weights are replicated across ranks
            parts.append((spec.name + ".W", wp.view(np.int16)))
            parts.append((spec.name + ".b", si.make_bias(seed, spec).view(np.int16)))
        offs, total = {}, 0
        for name, a in parts:
            offs[name] = total
            total += (a.size + 127) // 128 * 128
        self.host_all = torch.zeros(total, dtype=torch.int16).pin_memory()
        for name, a in parts:
            self.host_all[offs[name]: offs[name] + a.size].copy_(torch.from_numpy(np.ascontiguousarray(a).reshape(-1)))
        self.dev_all = self.host_all.to(device)
        view = lambda name, a: self.dev_all[offs[name]: offs[name] + a.size].view(a.shape)  # noqa: E731
        self.x = view("x", parts[0][1])
        self.lin = []
        for i, spec in enumerate(wl.linears):
            n_blocks = spec.n_out // spec.block
            e = {
                "spec": spec, "W": view(*parts[1 + 2 * i]), "b": view(*parts[2 + 2 * i]),
                "norms": torch.empty((n_blocks, spec.k_in), dtype=torch.float32, device=device),
                "gamma": torch.empty((n_blocks, spec.k_in), dtype=torch.float32, device=device),
                "penalty": torch.zeros(1, dtype=torch.float64, device=device),
                "pk": bsp.PackedMatrix.allocate(spec.n_out, spec.k_in, spec.block, bsp.ORIENT_C, device),
                "plan": view(*parts[1 + 2 * i]),      # in-place mode: W, masked where it is pruned, is its own execution layout
                "Y": torch.empty((wl.tokens, spec.n_out), dtype=torch.int16, device=device),
            }
            self.lin.append(e)
        self.kernels_per_step = 1 + len(self.lin)   # one weight-side launch for the batch, one GEMM per matrix

    def source(self, spec, outs):
        if spec.src == "x":
            return self.x
        if spec.src == "qkv_v":
            h = spec.k_in
            return outs["qkv"][:, 2 * h: 3 * h]
        return outs[spec.src]

    def step(self, gemm_events=None):
        """One pass of the path: one batched weight-side call for the four matrices (norms, gamma, penalty,
        keep flags, pack, plan: two launches), then the four GEMMs in order."""
        bsp, outs = self.bsp, {}
        if not hasattr(self, "jobs"):
            self.jobs = bsp.make_job_array([
                bsp.LayerJob(W=e["W"], out=e["pk"], threshold=0.0, norms=e["norms"], gamma_out=e["gamma"],
                             penalty=e["penalty"], plan=e["plan"]) for e in self.lin])
        bsp.bsp_prepare_batched(self.jobs, self.wl.linears[0].block, EPS, bsp.PEN_L2)
        for i, e in enumerate(self.lin):
            spec = e["spec"]
            src = self.source(spec, outs)
            if gemm_events is not None:
                gemm_events[i][0].record()
            bsp.bsp_linear_planned(e["plan"], spec.n_out, spec.k_in, spec.block, src, e["b"], int(spec.gelu), e["Y"])
            if gemm_events is not None:
                gemm_events[i][1].record()
            outs[spec.name.split(".")[1]] = e["Y"]
        return outs

    def upload_inputs(self):
        self.dev_all.copy_(self.host_all, non_blocking=True)

    def h2d_bytes(self):
        return self.host_all.numel() * 2

    def nonzero_flops(self):
        self.torch.cuda.synchronize()
        return [2 * self.wl.tokens * int(e["pk"].kept_weights.item()) for e in self.lin]


def rank_seed(seed: int, rank: int) -> int:
    """Seed of a rank's activations: every rank processes its own batch of tokens (weights are replicated)."""
    return seed + 1000 * rank


def reduce_max(values, device, world):
    """Element-wise maximum over ranks of a list of floats (the job takes as long as its slowest rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_throughput(world: int, flops_per_rank_step: int, steps: int, total_ms: float) -> float:
    """Whole-job TFLOP/s: all ranks' non-zero FLOPs over the slowest rank's time."""
    return world * flops_per_rank_step * steps / total_ms / 1e9


def dense_context(wl, device, iters=20):
    """torch.matmul (cuBLAS) bf16 on the same (tokens, N, K), L2 flushed: context, not part of the path."""
    import torch
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    out = {}
    for spec in wl.linears:
        a = torch.randn(wl.tokens, spec.k_in, device=device, dtype=torch.bfloat16)
        w = torch.randn(spec.n_out, spec.k_in, device=device, dtype=torch.bfloat16)
        for _ in range(3):
            torch.matmul(a, w.t())
        ms = []
        for _ in range(iters):
            flush.zero_()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            torch.matmul(a, w.t())
            e.record()
            torch.cuda.synchronize()
            ms.append(s.elapsed_time(e))
        t = statistics.median(ms)
        out[spec.name.split(".")[1]] = {"ms": round(t, 5), "dense_tflops": round(2 * wl.tokens * spec.n_out * spec.k_in / t / 1e9, 1)}
    return out


def stack_jobs(device):
    """The 72 weight matrices of a BERT-base encoder stack (d=16, about 3x) as one bsp_prepare_batched job array:
    (array, block height, weights, groups, kept groups, the LayerJob objects that own the buffers)."""
    import torch
    import paper_2009_08065_b200 as bsp
    d, rate = 16, 3.0
    shapes = [(768, 768)] * 48 + [(3072, 768)] * 12 + [(768, 3072)] * 12
    gen = torch.Generator(device=device)
    gen.manual_seed(si.DEFAULT_SEED)
    jobs, weights, groups, kept = [], 0, 0, 0
    for rows, cols in shapes:
        w = (torch.randn(rows, cols, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        keep = torch.rand(rows // d, cols, device=device, generator=gen) < (1.0 / rate)
        w = (w.view(rows // d, d, cols) * keep[:, None, :]).view(rows, cols).contiguous()
        pk = bsp.PackedMatrix.allocate(rows, cols, d, bsp.ORIENT_C, device)
        shape = (rows // d, cols)
        jobs.append(bsp.LayerJob(W=w, out=pk, threshold=0.0,
                                 norms=torch.empty(shape, dtype=torch.float32, device=device),
                                 gamma_out=torch.empty(shape, dtype=torch.float32, device=device),
                                 penalty=torch.zeros(1, dtype=torch.float64, device=device),
                                 plan=torch.empty(rows * cols * 2, dtype=torch.uint8, device=device)))
        weights += rows * cols
        groups += shape[0] * shape[1]
        kept += int(keep.sum().item())
    return bsp.make_job_array(jobs), d, weights, groups, kept, jobs


def weight_side_bandwidth(device, peaks, iters=10):
    """Achieved HBM GB/s of the weight-side kernels (bsp_prepare_batched: norms, gamma, penalty, keep flags,
    pack, plan) on the 72 weight matrices of a BERT-base encoder stack in one call, L2 flushed before each
    run.  A single 768x768 matrix is 1.2 MB, far too small to time against HBM on its own."""
    import torch
    import paper_2009_08065_b200 as bsp
    arr, d, weights, groups, kept, _keepalive = stack_jobs(device)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    ms = []
    for i in range(iters + 3):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        bsp.bsp_prepare_batched(arr, d, EPS, bsp.PEN_L2)
        b.record()
        torch.cuda.synchronize()
        if i >= 3:
            ms.append(a.elapsed_time(b))
    t = statistics.median(ms)
    # algorithmic bytes: W read once (2 B/weight); norms + gamma (4 B each) and a flag (1 B) per group;
    # kept values (2 B) and one index (4 B) per kept group; the execution layout (2 B/weight)
    alg = 2 * weights + 9 * groups + 2 * d * kept + 4 * kept + 2 * weights
    return {"kernels": "fused_stream_kernel (bsp_prepare_batched; W read once) + its clearing kernel",
            "workload": f"72 BERT-base weight matrices in one call, {weights * 2 / 1e6:.1f} MB of bf16 weights, d=16, ~3x",
            "ms": round(t, 4), "algorithmic_mb": round(alg / 1e6, 1), "achieved_gbs": round(alg / t / 1e6, 1),
            "peak_gbs": float(peaks["hbm_gbs"]), "frac": round(alg / t / 1e6 / float(peaks["hbm_gbs"]), 4),
            "l2": "flushed before each run"}


def retrain_step_bandwidth(device, peaks, iters=10):
    """Achieved HBM GB/s of bsp_masked_adam_step (Algorithm 2's retraining update with the mask applied, bf16 copy
    written) on as many weights as a BERT-base stack has (84.9 M, one [110592, 768] float32 matrix, d=16, ~3x)."""
    import torch
    import paper_2009_08065_b200 as bsp
    rows, cols, d = 110592, 768, 16
    gen = torch.Generator(device=device)
    gen.manual_seed(si.DEFAULT_SEED)
    W = torch.randn(rows, cols, device=device, generator=gen) * 0.02
    G = torch.randn(rows, cols, device=device, generator=gen) * 0.01
    M, V = torch.zeros_like(W), torch.zeros_like(W)
    keep = (torch.rand(rows // d, cols, device=device, generator=gen) < (1.0 / 3.0)).to(torch.uint8)
    Wb = torch.empty(rows, cols, dtype=torch.bfloat16, device=device)
    ms = []
    for i in range(iters + 3):          # 2.5 GB per launch: far larger than L2, no flush needed
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        bsp.bsp_masked_adam_step(W, G, M, V, keep, d, bsp.ORIENT_C, 3e-5, 0.9, 0.999, 1e-8, 0.0, i + 1, Wb)
        b.record()
        torch.cuda.synchronize()
        if i >= 3:
            ms.append(a.elapsed_time(b))
    t = statistics.median(ms)
    alg = rows * cols * 30 + (rows // d) * cols      # gradient, W, m, v in; W, m, v, bf16 copy out; one flag per group
    return {"kernel": "masked_adam_kernel (bsp_masked_adam_step)", "workload": f"{rows * cols / 1e6:.1f} M float32 weights, d=16, ~3x mask",
            "ms": round(t, 4), "algorithmic_mb": round(alg / 1e6, 1), "achieved_gbs": round(alg / t / 1e6, 1),
            "peak_gbs": float(peaks["hbm_gbs"]), "frac": round(alg / t / 1e6 / float(peaks["hbm_gbs"]), 4),
            "l2": "working set 2.5 GB per launch, larger than L2"}


def run_cuda(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    wl = workload()
    layer = LayerOnDevice(wl, si.DEFAULT_SEED, rank, device)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)

    # warm-up outside any graph (first calls set function attributes and the status word)
    for _ in range(max(args.warmup, 3)):
        layer.step()
    layer.bsp.bsp_linear_status()
    flops = layer.nonzero_flops()
    step_flops = sum(flops)

    # The step as a CUDA graph.  Two captures of the same call sequence: `graph` carries only the two
    # events that bracket the step and gives `value`; `graph_k` also brackets every GEMM launch and gives
    # the per-kernel durations of the roofline block (event nodes between kernels cost a few microseconds
    # each, so they are kept out of the step that is timed as a whole).
    ev = lambda: torch.cuda.Event(enable_timing=True, external=True)  # noqa: E731
    ev_step = (ev(), ev())
    ev_gemm = [(ev(), ev()) for _ in layer.lin]
    graph, graph_k = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ev_step[0].record()
        layer.step()
        ev_step[1].record()
    with torch.cuda.graph(graph_k):
        layer.step(gemm_events=ev_gemm)
    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        graph.replay()
        flush.zero_()
        graph_k.replay()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_ms, gemm_ms = [], [[] for _ in layer.lin]
    barrier()
    with ClockSampler(local_rank) as clocks:
        for _ in range(args.steps):
            flush.zero_()                  # untimed: evict the step's inputs from L2
            graph.replay()
            torch.cuda.synchronize()
            step_ms.append(ev_step[0].elapsed_time(ev_step[1]))
            flush.zero_()
            graph_k.replay()               # same step again, instrumented per kernel (not part of `value`)
            torch.cuda.synchronize()
            for i, (a, b) in enumerate(ev_gemm):
                gemm_ms[i].append(a.elapsed_time(b))
    barrier()
    layer.bsp.bsp_linear_status()
    total_ms = sum(step_ms)

    # the same step back to back without the flush: W, X and the intermediate outputs (about 100 MB) are
    # still in L2 from the previous step.  Context beside `value`, which is the flushed figure.
    w_s, w_e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph.replay()
    w_s.record()
    for _ in range(20):
        graph.replay()
    w_e.record()
    torch.cuda.synchronize()
    warm_ms = w_s.elapsed_time(w_e) / 20

    # end to end: pinned host inputs -> device, the step, result back to the host, every step.
    # (a) one step at a time: copy in, compute, copy out, in order on one stream;
    # (b) double-buffered, as a caller that feeds batches continuously would run it: two sets of device
    #     buffers and two captures of the step; the copies of a step overlap the kernels of its neighbours
    #     on separate streams.  Every step still moves all of its inputs and results inside the timed region.
    y_host = torch.empty_like(layer.lin[-1]["Y"], device="cpu").pin_memory()
    pen_host = torch.empty(len(layer.lin), dtype=torch.float64).pin_memory()
    e2e_ms = []
    e_s, e_e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(args.warmup + args.steps):
        barrier() if it == args.warmup else None
        e_s.record()
        layer.upload_inputs()
        graph.replay()
        y_host.copy_(layer.lin[-1]["Y"], non_blocking=True)
        for i, e in enumerate(layer.lin):
            pen_host[i:i + 1].copy_(e["penalty"], non_blocking=True)
        e_e.record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            e2e_ms.append(e_s.elapsed_time(e_e))
    e2e_serial_total_ms = sum(e2e_ms)

    layer_b = LayerOnDevice(wl, si.DEFAULT_SEED + 1, rank, device)       # the second set holds another batch
    layer_b.step()
    torch.cuda.synchronize()
    graph_b = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph_b):
        layer_b.step()
    sets = [(layer, graph), (layer_b, graph_b)]
    y_hosts = [y_host, torch.empty_like(y_host).pin_memory()]
    pen_hosts = [pen_host, torch.empty_like(pen_host).pin_memory()]
    s_main, s_in, s_out = torch.cuda.current_stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def pipelined(n_steps):
        ev_in = [torch.cuda.Event(), torch.cuda.Event()]
        ev_done = [torch.cuda.Event(), torch.cuda.Event()]
        ev_out = [torch.cuda.Event(), torch.cuda.Event()]
        for it in range(n_steps):
            k = it & 1
            lay, gr = sets[k]
            with torch.cuda.stream(s_in):
                if it >= 2:
                    s_in.wait_event(ev_done[k])        # the kernels of step it-2 have read this set's inputs
                lay.upload_inputs()
                ev_in[k].record(s_in)
            s_main.wait_event(ev_in[k])
            if it >= 2:
                s_main.wait_event(ev_out[k])           # the results of step it-2 have left this set's buffers
            gr.replay()
            ev_done[k].record(s_main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[k])
                y_hosts[k].copy_(lay.lin[-1]["Y"], non_blocking=True)
                for i, e in enumerate(lay.lin):
                    pen_hosts[k][i:i + 1].copy_(e["penalty"], non_blocking=True)
                ev_out[k].record(s_out)
        for k in range(min(2, n_steps)):
            s_main.wait_event(ev_out[k])

    pipelined(max(args.warmup, 3))
    barrier()
    e_s.record()
    pipelined(args.steps)
    e_e.record()
    torch.cuda.synchronize()
    e2e_total_ms = e_s.elapsed_time(e_e)
    barrier()
    layer_b.bsp.bsp_linear_status()

    total_ms, e2e_total_ms, e2e_serial_total_ms = reduce_max([total_ms, e2e_total_ms, e2e_serial_total_ms], device, world)

    if rank == 0:
        peaks, peak_src = measured_peaks()
        gemm_mean_ms = [statistics.mean(v) for v in gemm_ms]
        gemm_total = sum(gemm_mean_ms)
        achieved = step_flops / gemm_total / 1e9          # TFLOP/s over the four GEMM launches of a step
        peak = float(peaks["bf16_tflops"])
        value = job_throughput(world, step_flops, args.steps, total_ms)
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(total_ms / args.steps, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": wl.name + " (one BERT-base encoder layer: QKV, attn-out, FFN-up+GELU, FFN-down; "
                            "tokens per GPU 4096; 16-row blocks; 3.0x compression)",
                "step": "bsp_prepare_batched (norms+gamma+penalty, keep flags, pack, plan of the 4 matrices: a clearing kernel and one kernel that reads W once) "
                        "then the 4 GEMMs in sequence (bsp_linear_planned; the single chained launch bsp_linear_chain measured "
                        "8 % slower on this workload); one CUDA graph",
                "l2": f"flushed between steps by writing {L2_FLUSH_BYTES >> 20} MiB",
                "parallelism": "token split, replicated weights, no collective" if world > 1 else "single GPU",
                "nonzero_gflop_per_step_per_gpu": round(step_flops / 1e9, 3),
            },
            "percent_of_bf16_peak": round(100 * value / world / peak, 2),
            "warm_l2": {"ms_per_step": round(warm_ms, 5), "value": round(step_flops / warm_ms / 1e9, 2), "unit": UNIT,
                        "how": "rank 0, 20 steps back to back, no flush between them"},
            "e2e": {"value": round(job_throughput(world, step_flops, args.steps, e2e_total_ms), 3), "unit": UNIT,
                    "h2d_bytes_per_step": layer.h2d_bytes(),
                    "d2h_bytes_per_step": y_host.numel() * 2 + pen_host.numel() * 8,
                    "how": "double-buffered: two sets of device buffers, copies on their own streams overlap the "
                           "kernels of the neighbouring steps; every step copies all its inputs in and its result out",
                    "one_step_at_a_time": round(job_throughput(world, step_flops, len(e2e_ms), e2e_serial_total_ms), 3)},
            "gpu_launches": 2 * layer.kernels_per_step * args.steps,
            "clocks": clocks.summary(),
            "roofline": {
                "kernel": "linear_tc_kernel (bsp_linear_planned), the four launches of a step",
                "bound": "tensor", "achieved": round(achieved, 2), "peak": peak, "unit": "TFLOP/s",
                "frac": round(achieved / peak, 4),
                # dram__bytes_read.sum + dram__bytes_write.sum of the four launches, one ncu capture each
                # (profiles/linear_tc_kernel_bert_base_T4096.md); Y is still in L2 when each kernel ends
                "traffic": 58.31e6, "algorithmic_bytes": sum(
                    2 * wl.tokens * sp.k_in + 2 * sp.n_out * sp.k_in + 2 * wl.tokens * sp.n_out + 2 * sp.n_out
                    for sp in wl.linears),
                "peak_source": f"bf16_tflops burst, {peak_src}",
                "per_launch": {e["spec"].name.split(".")[1]: {
                    "ms": round(gemm_mean_ms[i], 5), "nonzero_tflops": round(flops[i] / gemm_mean_ms[i] / 1e9, 1)}
                    for i, e in enumerate(layer.lin)},
            },
        }
        if world == 1:
            line["weight_side_hbm"] = weight_side_bandwidth(device, peaks)
            line["retrain_step_hbm"] = retrain_step_bandwidth(device, peaks)
            line["dense_gemm_context"] = dense_context(wl, device)
            line["cpu_baseline"] = oracle_baseline(wl, reps=3)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands
# ------------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_step(wl, inputs):
    """The same step on the oracle: norms, gamma, penalty, keep flags, pack, masked dense product."""
    from oracle import bsp_oracle as O
    x, mats = inputs
    kept = 0
    for spec, wp, b, xin in mats:
        n = O.group_norms(wp, spec.block, "C")
        g = O.gamma_update(n, EPS)
        O.penalty_l2(n, g)
        keep = O.keep_flags(wp, spec.block, "C", 0.0)
        O.pack(wp, keep, spec.block, "C")
        O.linear_masked_dense(xin, wp, O.mask_of(wp), b, int(spec.gelu))
        kept += spec.block * int(keep.sum())
    return kept


def oracle_inputs(wl, seed, tokens):
    x = si.make_activations(seed, "layer_in", tokens, wl.linears[0].k_in)
    mats = []
    for spec in wl.linears:
        wp, _ = si.make_pruned_weight(seed, spec)
        # each linear gets fresh N(0,1) activations of its input width (the oracle is not chained)
        xin = x if spec.src == "x" else si.make_activations(seed, spec.name, tokens, spec.k_in)
        mats.append((spec, wp, si.make_bias(seed, spec), xin))
    return x, mats


def oracle_baseline(wl, reps):
    inputs = oracle_inputs(wl, si.DEFAULT_SEED, wl.tokens)
    oracle_step(wl, inputs)                                  # first call pays imports and page faults
    t0 = time.perf_counter()
    for _ in range(reps):
        kept = oracle_step(wl, inputs)
    dt = (time.perf_counter() - t0) / reps
    return {"value": round(2 * wl.tokens * kept / dt / 1e12, 5), "unit": UNIT, "cores": oracle_threads(),
            "kind": "oracle", "seconds_per_step": round(dt, 4),
            "sample": f"the full workload ({wl.tokens} tokens, 4 matrices), {reps} steps after one untimed step"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload()
    inputs = oracle_inputs(wl, si.DEFAULT_SEED, wl.tokens)
    steps = min(args.steps, 20)                              # about 1 s each: keeps the run within minutes
    warm = min(max(args.warmup, 1), 3)
    for _ in range(warm):
        kept = oracle_step(wl, inputs)
    t0 = time.perf_counter()
    for _ in range(steps):
        kept = oracle_step(wl, inputs)
    dt = time.perf_counter() - t0
    value = round(2 * wl.tokens * kept * steps / dt / 1e12, 5)
    sample = f"the full workload ({wl.tokens} tokens, 4 matrices) per step; {steps} timed steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": warm, "ms_per_step": round(1e3 * dt / steps, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name + " on the CPU oracle (numpy float64), rank 0 only"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def run_case(args):
    """A handful of launches of one call, for profilers (no timing, no JSON):
    --case qkv|attn_out|ffn_up|ffn_down runs that linear's GEMM on the bench workload, --case prepare the batched
    weight-side call on its four matrices, --case prepare_stack the same call on the 72 matrices of a BERT-base
    stack (inputs larger than L2), --case gather the gathering linear kernel on a BERT-large FFN-up point
    (16384 tokens, 1024 -> 4096, 64-row blocks, 5x)."""
    import torch
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    if args.case == "prepare_stack":
        import paper_2009_08065_b200 as bsp
        stack = stack_jobs(device)          # keeps the buffers alive
        arr, d = stack[0], stack[1]
        for _ in range(3):
            bsp.bsp_prepare_batched(arr, d, EPS, bsp.PEN_L2)
        bsp.bsp_linear_status()
        print("case prepare_stack: 3 calls done")
        return
    if args.case == "gather":
        import paper_2009_08065_b200 as bsp
        T, N, K, d, c = 16384, 4096, 1024, 64, 5.0
        gen = torch.Generator(device=device)
        gen.manual_seed(si.DEFAULT_SEED)
        X = torch.randn(T, K, device=device, generator=gen).to(torch.bfloat16)
        XT = torch.empty(K, T, dtype=torch.bfloat16, device=device)
        bsp.bsp_transpose(X, XT)
        Wd = (torch.randn(N, K, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        keep = torch.zeros(N // d, K, dtype=torch.bool, device=device)
        keep.scatter_(1, torch.rand(N // d, K, device=device, generator=gen).topk(int(round(K / c)), dim=1).indices, True)
        W = (Wd.view(N // d, d, K) * keep[:, None, :]).view(N, K).contiguous()
        pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, device)
        bsp.bsp_prune_pack(W, pk, 0.0)
        gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=device)
        bsp.bsp_linear_gather_plan(pk, gplan)
        bias = (torch.randn(N, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        Y = torch.empty(T, N, dtype=torch.bfloat16, device=device)
        for _ in range(3):
            bsp.bsp_linear_gathered(gplan, N, K, d, XT, bias, 1, Y)
        bsp.bsp_linear_status()
        print("case gather: 3 launches done")
        return
    layer = LayerOnDevice(workload(), si.DEFAULT_SEED, 0, device)
    layer.step()
    torch.cuda.synchronize()
    bsp = layer.bsp
    for _ in range(4):
        if args.case == "prepare":
            bsp.bsp_prepare_batched(layer.jobs, layer.wl.linears[0].block, EPS, bsp.PEN_L2)
        else:
            outs = {"qkv": layer.lin[0]["Y"], "attn_out": layer.lin[1]["Y"], "ffn_up": layer.lin[2]["Y"]}
            e = next(e for e in layer.lin if e["spec"].name.endswith("." + args.case))
            spec = e["spec"]
            bsp.bsp_linear_planned(e["plan"], spec.n_out, spec.k_in, spec.block, layer.source(spec, outs), e["b"],
                                   int(spec.gelu), e["Y"])
    bsp.bsp_linear_status()
    print(f"case {args.case}: 4 launches done")


def run_sweep(args):
    """The BERT-large sweep (hidden 1024, FFN 4096, tokens 32768 by default): compression 1.5/2/3/5/8 x block height
    8/16/32/64 (and 128) on the four linear shapes.  For every point: the zero-expanded dense route (bsp_linear_planned), the
    gathering kernel (bsp_linear_gathered, block heights it takes; X transposed beforehand, that copy timed
    separately once per input width), and torch.matmul on the dense shape as context.  L2 is flushed (256 MiB
    written) before every timed launch; medians of `--steps` launches.  One JSON line per point."""
    import torch
    import paper_2009_08065_b200 as bsp
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peaks, _ = measured_peaks()
    peak = float(peaks["bf16_tflops"])
    T = args.sweep_tokens
    iters = max(3, min(args.steps, 20))
    shapes = [("qkv", 3072, 1024, 0), ("attn_out", 1024, 1024, 0), ("ffn_up", 4096, 1024, 1), ("ffn_down", 1024, 4096, 0)]
    if args.sweep_shapes:
        shapes = [sh for sh in shapes if sh[0] in args.sweep_shapes.split(",")]
    gen = torch.Generator(device=device)
    gen.manual_seed(si.DEFAULT_SEED)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)

    def timed(fn):
        ms = []
        for i in range(iters + 2):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if i >= 2:
                ms.append(a.elapsed_time(b))
        return statistics.median(ms)

    for name, N, K, act in shapes:
        X = torch.randn(T, K, device=device, generator=gen).to(torch.bfloat16)
        XT = torch.empty(K, T, dtype=torch.bfloat16, device=device)
        t_tr = timed(lambda: bsp.bsp_transpose(X, XT))
        bias = (torch.randn(N, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        Y = torch.empty(T, N, dtype=torch.bfloat16, device=device)
        Yg = torch.empty(T, N, dtype=torch.bfloat16, device=device)
        Wd = (torch.randn(N, K, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        t_dense = timed(lambda: torch.matmul(X, Wd.t()))
        for d in (8, 16, 32, 64, 128):        # 128 is beyond the named grid: it shows where the gathering kernel is heading
            for c in (1.5, 2.0, 3.0, 5.0, 8.0):
                kc = int(round(K / c))
                scores = torch.rand(N // d, K, device=device, generator=gen)
                keep = torch.zeros(N // d, K, dtype=torch.bool, device=device)
                keep.scatter_(1, scores.topk(kc, dim=1).indices, True)
                W = (Wd.view(N // d, d, K) * keep[:, None, :]).view(N, K).contiguous()
                pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, device)
                bsp.bsp_prune_pack(W, pk, 0.0)
                plan = torch.empty(bsp.bsp_linear_plan_bytes(N, K, d), dtype=torch.uint8, device=device)
                bsp.bsp_linear_plan(pk, plan)
                nz = 2.0 * T * d * kc * (N // d)
                t_plan = timed(lambda: bsp.bsp_linear_planned(plan, N, K, d, X, bias, act, Y))
                point = {"sweep": "bert_large", "shape": name, "tokens": T, "n_out": N, "k_in": K, "block": d,
                         "compression": c, "kept_per_block": kc, "nonzero_gflop": round(nz / 1e9, 2),
                         "dense_route_ms": round(t_plan, 4), "dense_route_nonzero_tflops": round(nz / t_plan / 1e9, 1),
                         "torch_dense_ms": round(t_dense, 4), "torch_dense_tflops": round(2.0 * T * N * K / t_dense / 1e9, 1),
                         "transpose_ms": round(t_tr, 4)}
                best = nz / t_plan / 1e9
                if d in (16, 32, 64, 128):
                    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=device)
                    bsp.bsp_linear_gather_plan(pk, gplan)
                    t_g = timed(lambda: bsp.bsp_linear_gathered(gplan, N, K, d, XT, bias, act, Yg))
                    diff = (Y.float() - Yg.float()).abs().max().item()
                    point.update({"gather_ms": round(t_g, 4), "gather_nonzero_tflops": round(nz / t_g / 1e9, 1),
                                  "gather_vs_dense_route": round(t_plan / t_g, 3), "max_abs_diff_between_routes": diff})
                    best = max(best, nz / t_g / 1e9)
                    del gplan
                point["best_percent_of_bf16_peak"] = round(100.0 * best / peak, 2)
                bsp.bsp_linear_status()
                print(json.dumps(point), flush=True)
                del plan, pk, W, keep, scores


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--case", choices=["qkv", "attn_out", "ffn_up", "ffn_down", "prepare", "prepare_stack", "gather"], default=None,
                    help="run a few launches of one call for a profiler and exit")
    ap.add_argument("--sweep", choices=["bert_large"], default=None,
                    help="time the BERT-large compression x block-height grid and print one JSON line per point")
    ap.add_argument("--sweep-tokens", type=int, default=32768)
    ap.add_argument("--sweep-shapes", default=None, help="comma-separated subset of qkv,attn_out,ffn_up,ffn_down")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
