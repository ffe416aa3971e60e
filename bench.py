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
        self.weight_side_launches = 2               # a small clearing kernel and the one-pass kernel
        self.kernels_per_step = self.weight_side_launches + len(self.lin)

    def source(self, spec, outs):
        if spec.src == "x":
            return self.x
        if spec.src == "qkv_v":
            h = spec.k_in
            return outs["qkv"][:, 2 * h: 3 * h]
        return outs[spec.src]

    def step(self, n_linears=None):
        """One pass of the path: one batched weight-side call for the four matrices (norms, gamma, penalty,
        keep flags, pack; W, already zero where it is pruned, is its own execution layout: in-place mode), then the
        four GEMMs in order.  `n_linears` < 4 runs only the first few GEMMs (the prefixes that give each launch's
        share of the step)."""
        bsp = self.bsp
        outs = {e["spec"].name.split(".")[1]: e["Y"] for e in self.lin}   # (a prefix may start from earlier outputs)
        if not hasattr(self, "jobs"):
            self.jobs = bsp.make_job_array([
                bsp.LayerJob(W=e["W"], out=e["pk"], threshold=0.0, norms=e["norms"], gamma_out=e["gamma"],
                             penalty=e["penalty"], plan=e["plan"]) for e in self.lin])
        bsp.bsp_prepare_batched(self.jobs, self.wl.linears[0].block, EPS, bsp.PEN_L2)
        for i, e in enumerate(self.lin[:n_linears]):
            spec = e["spec"]
            # the weights of every linear but the first were finished before the kernel that precedes it began
            algo = bsp.LINEAR_AUTO | (bsp.LINEAR_PLAN_STABLE if i > 0 else 0)
            bsp.bsp_linear_planned_ex(e["plan"], spec.n_out, spec.k_in, spec.block, self.source(spec, outs), e["b"],
                                      int(spec.gelu), e["Y"], algo)
        return outs

    def upload_inputs(self, activations_only=False):
        n = self.x.numel() if activations_only else self.host_all.numel()       # x is the first view of the buffer
        self.dev_all[:n].copy_(self.host_all[:n], non_blocking=True)

    def h2d_bytes(self, activations_only=False):
        return (self.x.numel() if activations_only else self.host_all.numel()) * 2

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
                                 plan=w))          # in-place mode: W, zero where pruned, is its own execution layout
        weights += rows * cols
        groups += shape[0] * shape[1]
        kept += int(keep.sum().item())
    return bsp.make_job_array(jobs), d, weights, groups, kept, jobs


def weight_side_bandwidth(device, peaks, iters=10):
    """Achieved HBM GB/s of the weight-side kernels (bsp_prepare_batched: norms, gamma, penalty, keep flags,
    pack; in-place mode, so no separate execution layout is written) on the 72 weight matrices of a BERT-base
    encoder stack in one call, L2 flushed before each run.  A single 768x768 matrix is 1.2 MB, far too small to
    time against HBM on its own."""
    import torch
    import paper_2009_08065_b200 as bsp
    arr, d, weights, groups, kept, _keepalive = stack_jobs(device)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    def timed(pen):
        ms = []
        for i in range(iters + 3):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            bsp.bsp_prepare_batched(arr, d, EPS, pen)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                ms.append(a.elapsed_time(b))
        return statistics.mean(ms)
    t = timed(bsp.PEN_L2)                    # the paper's form: sum gamma ||W_g||, gamma = 1 / (||W_g|| + eps)
    t_sq = timed(bsp.PEN_L2SQ)               # the squared-norm form: the same pass, a different last step per group
    # algorithmic bytes: W read once (2 B/weight); norms + gamma (4 B each) and a flag (1 B) per group;
    # kept values (2 B) and one index (4 B) per kept group.  No execution layout: W already holds zeros in the
    # pruned groups, so in-place mode writes nothing into it.
    alg = 2 * weights + 9 * groups + 2 * d * kept + 4 * kept
    return {"kernels": "fused_stream_kernel (bsp_prepare_batched; W read once) + its clearing kernel",
            "workload": f"72 BERT-base weight matrices in one call, {weights * 2 / 1e6:.1f} MB of bf16 weights, d=16, ~3x",
            "ms": round(t, 4), "ms_squared_norm_penalty": round(t_sq, 4),
            "algorithmic_mb": round(alg / 1e6, 1), "achieved_gbs": round(alg / t / 1e6, 1),
            "peak_gbs": float(peaks["hbm_gbs"]), "frac": round(alg / t / 1e6 / float(peaks["hbm_gbs"]), 4),
            "algorithmic_bytes_formula": "2/weight (W once) + 9/group (norm, gamma, flag) + (2d + 4)/kept group (values, index)",
            "plan_bytes": 0, "plan_note": "in-place mode: no separate execution layout is written",
            "l2": "flushed before each run", "timing": f"mean of {iters} launches"}


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


def _timed_graph(torch, fn, flush, iters, cold):
    """Mean milliseconds of `fn` captured as a CUDA graph; cold = L2 flushed before every replay, else back to back."""
    a, b = torch.cuda.Event(enable_timing=True, external=True), torch.cuda.Event(enable_timing=True, external=True)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        a.record()
        fn()
        b.record()
    ms = []
    for i in range(iters + 2):
        if cold:
            flush.zero_()
        g.replay()
        torch.cuda.synchronize()
        if i >= 2:
            ms.append(a.elapsed_time(b))
    return statistics.mean(ms)


def _stack_report(name, tokens, mats, t_full, t_gemm, peaks, note):
    """Figures of a chained stack: mats = [(n_out, k_in, block, kept_weights)], t_* = {"cold": ms, "warm": ms}."""
    peak, hbm = float(peaks["bf16_tflops"]), float(peaks["hbm_gbs"])
    flops = [2 * tokens * kw for (_n, _k, _d, kw) in mats]
    byts = [2 * tokens * k + 2 * kw + 4 * (kw // d) + 2 * tokens * n + 2 * n for (n, k, d, kw) in mats]
    t_roof = sum(max(f / peak / 1e9, b / hbm / 1e6) for f, b in zip(flops, byts))     # ms, min(tensor, HBM) roofline
    total = sum(n * k for (n, k, _d, _kw) in mats)
    kept = sum(kw for (*_x, kw) in mats)
    out = {"workload": name, "tokens": tokens, "matrices": len(mats), "nonzero_gflop": round(sum(flops) / 1e9, 2),
           "compression": round(total / kept, 4), "algorithmic_mb": round(sum(byts) / 1e6, 1),
           "roofline_ms": round(t_roof, 4), "note": note}
    for label, t in (("gemms", t_gemm), ("with_weight_side", t_full)):
        out[label] = {
            k: {"ms": round(v, 4), "nonzero_tflops": round(sum(flops) / v / 1e9, 1),
                "percent_of_bf16_peak": round(100 * sum(flops) / v / 1e9 / peak, 2),
                "frac_of_min_tensor_hbm_roofline": round(t_roof / v, 4) if label == "gemms" else None}
            for k, v in t.items()}
    return out


def stack_72_matrices(device, peaks, iters=5):
    """The 72 weight matrices of a BERT-base encoder stack (12 layers of Q, K, V, O, FFN-up, FFN-down), 4096 tokens,
    16-row blocks, per-matrix rates drawn from U(3, 7) and scaled to 5.0x overall, layer outputs chained (O reads V's
    output, FFN-up reads O's through GELU, FFN-down reads FFN-up's, the next layer reads FFN-down's)."""
    import torch
    import paper_2009_08065_b200 as bsp
    T, H, F, d = 4096, 768, 3072, 16
    rates = si.bert_base_stack_rates(si.DEFAULT_SEED)
    gen = torch.Generator(device=device)
    gen.manual_seed(si.DEFAULT_SEED)
    shapes = [("q", H, H, 0), ("k", H, H, 0), ("v", H, H, 0), ("o", H, H, 0), ("up", F, H, 1), ("down", H, F, 0)]
    x0 = torch.randn(T, H, device=device, generator=gen).to(torch.bfloat16)
    bufs = {nm: torch.empty(T, n, dtype=torch.bfloat16, device=device) for nm, n, _k, _a in shapes}
    nxt = torch.empty(T, H, dtype=torch.bfloat16, device=device)
    layers, jobs, mats = [], [], []
    for l in range(12):
        ops = []
        for j, (nm, n, k, act) in enumerate(shapes):
            kc = int(round(k / rates[l][j]))
            w = (torch.randn(n, k, device=device, generator=gen) * 0.02).to(torch.bfloat16)
            keep = torch.zeros(n // d, k, dtype=torch.bool, device=device)
            keep.scatter_(1, torch.rand(n // d, k, device=device, generator=gen).topk(kc, dim=1).indices, True)
            w = (w.view(n // d, d, k) * keep[:, None, :]).view(n, k).contiguous()
            bias = (torch.randn(n, device=device, generator=gen) * 0.02).to(torch.bfloat16)
            pk = bsp.PackedMatrix.allocate(n, k, d, bsp.ORIENT_C, device)
            g = (n // d, k)
            jobs.append(bsp.LayerJob(W=w, out=pk, threshold=0.0, norms=torch.empty(g, dtype=torch.float32, device=device),
                                     gamma_out=torch.empty(g, dtype=torch.float32, device=device),
                                     penalty=torch.zeros(1, dtype=torch.float64, device=device), plan=w))
            ops.append((nm, w, bias, n, k, act))
            mats.append((n, k, d, d * kc * (n // d)))
        layers.append(ops)
    arr = bsp.make_job_array(jobs)

    def gemms():
        src, first = x0, True
        for l, ops in enumerate(layers):
            out_down = nxt if l % 2 == 0 else bufs["down"]
            for nm, w, bias, n, k, act in ops:
                inp = {"q": src, "k": src, "v": src, "o": bufs["v"], "up": bufs["o"], "down": bufs["up"]}[nm]
                dst = out_down if nm == "down" else bufs[nm]
                bsp.bsp_linear_planned_ex(w, n, k, d, inp, bias, act, dst, 0 if first else bsp.LINEAR_PLAN_STABLE)
                first = False
            src = out_down

    def full():
        bsp.bsp_prepare_batched(arr, d, EPS, bsp.PEN_L2)
        gemms()

    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    full()
    bsp.bsp_linear_status()
    t_gemm = {"cold": _timed_graph(torch, gemms, flush, iters, True), "warm": _timed_graph(torch, gemms, flush, iters, False)}
    t_full = {"cold": _timed_graph(torch, full, flush, iters, True), "warm": _timed_graph(torch, full, flush, iters, False)}
    bsp.bsp_linear_status()
    return _stack_report("BERT-base stack, 72 matrices, 5.0x overall, d=16", T, mats, t_full, t_gemm, peaks,
                         "cold = L2 flushed before each pass over the stack (activations then stay in L2 from one linear to the next); "
                         "warm = passes back to back (170 MB of weights do not fit the 126 MB L2); one CUDA graph per pass")


def stack_distil(device, peaks, iters=5):
    """DistilBERT-shaped stack: 6 layers (fused QKV, O, FFN-up, FFN-down), 8192 tokens, 32-row blocks, heavy-tailed
    weights (Student-t, 3 degrees of freedom, std 0.02), every matrix through the real pipeline in every pass:
    bsp_percentile_threshold_batched (1.79x) -> bsp_prepare_batched with that device threshold (norms, gamma, penalty, flags,
    pack, W masked in place) -> the linear layer; kept counts differ from block to block."""
    import torch
    import paper_2009_08065_b200 as bsp
    wl = si.distil_stack()
    T, d = wl.tokens, wl.linears[0].block
    gen = torch.Generator(device=device)
    gen.manual_seed(si.DEFAULT_SEED + 4)
    x0 = torch.randn(T, 768, device=device, generator=gen).to(torch.bfloat16)
    ops, jobs = [], []
    for spec in wl.linears:
        n, k = spec.n_out, spec.k_in
        z = torch.randn(n, k, device=device, generator=gen)
        chi = (torch.randn(3, n, k, device=device, generator=gen) ** 2).sum(0) / 3.0
        w0 = (z / chi.sqrt() * (0.02 / 3 ** 0.5)).to(torch.bfloat16)
        w = w0.clone()
        thr = torch.zeros(1, dtype=torch.float32, device=device)
        pk = bsp.PackedMatrix.allocate(n, k, d, bsp.ORIENT_C, device)
        g = (n // d, k)
        jobs.append(bsp.LayerJob(W=w, out=pk, threshold=0.0, threshold_dev=thr,
                                 norms=torch.empty(g, dtype=torch.float32, device=device),
                                 gamma_out=torch.empty(g, dtype=torch.float32, device=device),
                                 penalty=torch.zeros(1, dtype=torch.float64, device=device), plan=w))
        ops.append({"spec": spec, "w0": w0, "w": w, "thr": thr, "pk": pk,
                    "bias": (torch.randn(n, device=device, generator=gen) * 0.02).to(torch.bfloat16),
                    "y": torch.empty(T, n, dtype=torch.bfloat16, device=device)})
    arr = bsp.make_job_array(jobs)

    def restore():
        for o in ops:
            o["w"].copy_(o["w0"])

    rates = [o["spec"].rate for o in ops]

    def weight_side():
        bsp.bsp_percentile_threshold_batched(arr, d, rates)
        bsp.bsp_prepare_batched(arr, d, EPS, bsp.PEN_L2)

    def gemms():
        outs = {}
        for i, o in enumerate(ops):
            spec = o["spec"]
            layer_tag, nm = spec.name.split(".")
            if spec.src == "x":
                src = x0
            elif spec.src == "qkv_v":
                src = outs[layer_tag + ".qkv"][:, 2 * spec.k_in: 3 * spec.k_in]
            elif "." in spec.src:
                src = outs[spec.src]
            else:
                src = outs[layer_tag + "." + spec.src]
            bsp.bsp_linear_planned_ex(o["w"], spec.n_out, spec.k_in, d, src, o["bias"], int(spec.gelu), o["y"],
                                      bsp.LINEAR_PLAN_STABLE if i > 0 else 0)
            outs[spec.name] = o["y"]

    def full():
        restore()            # the pass prunes the unpruned weights every time (this copy is part of the timed pass)
        weight_side()
        gemms()

    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    full()
    bsp.bsp_linear_status()
    torch.cuda.synchronize()
    mats = [(o["spec"].n_out, o["spec"].k_in, d, int(o["pk"].kept_weights.item())) for o in ops]
    t_gemm = {"cold": _timed_graph(torch, gemms, flush, iters, True), "warm": _timed_graph(torch, gemms, flush, iters, False)}
    t_full = {"cold": _timed_graph(torch, full, flush, iters, True), "warm": _timed_graph(torch, full, flush, iters, False)}
    bsp.bsp_linear_status()
    return _stack_report("DistilBERT-shaped stack, 24 matrices (fused QKV), 1.79x by per-matrix percentile, d=32, Student-t weights",
                         T, mats, t_full, t_gemm, peaks,
                         "with_weight_side = restore the unpruned weights (a device copy), percentile threshold, norms/gamma/penalty/"
                         "flags/pack with W masked in place, then the linears; gemms = the linears alone on the masked weights")


def bert_large_grid(device, peaks, tokens, iters, shapes_filter=None, emit=None):
    """The BERT-large grid (hidden 1024, FFN 4096): compression 1.5/2/3/5/8 x block height 8/16/32/64 on the four linear
    shapes; per point the zero-expanded route (bsp_linear_planned) and, where the block height allows, the gathering
    kernel (bsp_linear_gathered on transposed activations), each launch after an L2 flush, mean of `iters`."""
    import torch
    import paper_2009_08065_b200 as bsp
    peak = float(peaks["bf16_tflops"])
    T = tokens
    shapes = [("qkv", 3072, 1024, 0), ("attn_out", 1024, 1024, 0), ("ffn_up", 4096, 1024, 1), ("ffn_down", 1024, 4096, 0)]
    if shapes_filter:
        shapes = [sh for sh in shapes if sh[0] in shapes_filter]
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
        return statistics.mean(ms)

    points = []
    for name, N, K, act in shapes:
        X = torch.randn(T, K, device=device, generator=gen).to(torch.bfloat16)
        XT = torch.empty(K, T, dtype=torch.bfloat16, device=device)
        t_tr = timed(lambda: bsp.bsp_transpose(X, XT))
        bias = (torch.randn(N, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        Y = torch.empty(T, N, dtype=torch.bfloat16, device=device)
        Yg = torch.empty(T, N, dtype=torch.bfloat16, device=device)
        Wd = (torch.randn(N, K, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        t_dense = timed(lambda: torch.matmul(X, Wd.t()))
        for d in (8, 16, 32, 64):
            for c in (1.5, 2.0, 3.0, 5.0, 8.0):
                kc = int(round(K / c))
                keep = torch.zeros(N // d, K, dtype=torch.bool, device=device)
                keep.scatter_(1, torch.rand(N // d, K, device=device, generator=gen).topk(kc, dim=1).indices, True)
                W = (Wd.view(N // d, d, K) * keep[:, None, :]).view(N, K).contiguous()      # masked W = its own execution layout
                nz = 2.0 * T * d * kc * (N // d)
                t_plan = timed(lambda: bsp.bsp_linear_planned(W, N, K, d, X, bias, act, Y))
                t_plan_t = None
                if d == 64 and c == 8.0:     # the epilogue that hands transposed activations to a gathering next layer
                    YT = torch.empty(N, T, dtype=torch.bfloat16, device=device)
                    t_plan_t = timed(lambda: bsp.bsp_linear_planned_ex(W, N, K, d, X, bias, act, YT, bsp.LINEAR_OUT_TRANSPOSED))
                    del YT
                point = {"shape": name, "tokens": T, "n_out": N, "k_in": K, "block": d, "compression": c,
                         "nonzero_gflop": round(nz / 1e9, 2), "dense_route_ms": round(t_plan, 4),
                         "dense_route_nonzero_tflops": round(nz / t_plan / 1e9, 1),
                         "torch_dense_ms": round(t_dense, 4), "transpose_ms": round(t_tr, 4)}
                if t_plan_t is not None:
                    point["dense_route_transposed_output_ms"] = round(t_plan_t, 4)
                best, route, auto = nz / t_plan / 1e9, "zero-expanded", "zero-expanded"
                if d in (16, 32, 64, 128):
                    pk = bsp.PackedMatrix.allocate(N, K, d, bsp.ORIENT_C, device)
                    bsp.bsp_prune_pack(W, pk, 0.0)
                    gplan = torch.empty(bsp.bsp_linear_gather_plan_bytes(N, K, d), dtype=torch.uint8, device=device)
                    bsp.bsp_linear_gather_plan(pk, gplan)
                    t_g = timed(lambda: bsp.bsp_linear_gathered(gplan, N, K, d, XT, bias, act, Yg))
                    point.update({"gather_ms": round(t_g, 4), "gather_nonzero_tflops": round(nz / t_g / 1e9, 1),
                                  # a first layer whose input arrives row-major pays the transposing pass once; later
                                  # layers of a chain get their input transposed from the previous layer's epilogue
                                  "gather_incl_transpose_nonzero_tflops": round(nz / (t_g + t_tr) / 1e9, 1),
                                  "max_abs_diff_between_routes": (Y.float() - Yg.float()).abs().max().item()})
                    if nz / t_g / 1e9 > best:
                        best, route = nz / t_g / 1e9, "gathered"
                    # what the library's own choice gives when both layouts of weights and activations are at hand
                    call = bsp.make_linear_call(N, K, d, T, plan=W, gplan=gplan, kept_weights=d * kc * (N // d), X=X, XT=XT,
                                                bias=bias, act=act, Y=Y)
                    auto = "gathered" if bsp.bsp_linear_route(call) == bsp.ROUTE_GATHERED else "zero-expanded"
                    del gplan, pk
                t_auto = t_g if auto == "gathered" else t_plan
                point.update({"auto_route": auto, "auto_nonzero_tflops": round(nz / t_auto / 1e9, 1),
                              "auto_vs_best": round((nz / t_auto / 1e9) / best, 4)})
                f, b = nz, 2 * T * K + 2 * N * kc + 4 * (N // d) * kc + 2 * T * N + 2 * N
                t_roof = max(f / peak / 1e9, b / float(peaks["hbm_gbs"]) / 1e6)
                point.update({"best_route": route, "best_nonzero_tflops": round(best, 1),
                              "best_percent_of_bf16_peak": round(100.0 * best / peak, 2),
                              "frac_of_min_tensor_hbm_roofline": round(t_roof / (nz / best / 1e9), 4)})
                bsp.bsp_linear_status()
                points.append(point)
                if emit:
                    emit(point)
                del W, keep
    return points


def other_workloads(device, peaks, args):
    """Figures of the workloads that are not the bench line's own: outside its timed region, fewer repetitions."""
    out = {"bert_base_stack_72": stack_72_matrices(device, peaks), "distil_stack": stack_distil(device, peaks)}
    pts = bert_large_grid(device, peaks, 32768, 3)
    out["bert_large_grid"] = {
        "tokens": 32768, "how": "each launch after an L2 flush (cold), mean of 3; a launch's operands and output are 136-340 MB, more than the 126 MB L2, "
                                "so a back-to-back figure would be the same; cells = [best non-zero TFLOP/s, % of bf16 peak, route, what bsp_linear_route picks / best]; "
                                "the gathering kernel's figures take the transposed activations as given (see transpose_ms)",
        "cells": {f"{p['shape']}/d{p['block']}/c{p['compression']:g}": [p["best_nonzero_tflops"], p["best_percent_of_bf16_peak"],
                                                                       "g" if p["best_route"] == "gathered" else "z", p["auto_vs_best"]] for p in pts},
        "auto_route_worst_vs_best": min(p["auto_vs_best"] for p in pts),
        "transpose_ms": {p["shape"]: p["transpose_ms"] for p in pts},
        "zero_expanded_ms_row_major_vs_transposed_output": {p["shape"]: [p["dense_route_ms"], p["dense_route_transposed_output_ms"]]
                                                            for p in pts if "dense_route_transposed_output_ms" in p},
        "gathered_incl_transpose_of_x": {f"{p['shape']}/d{p['block']}/c{p['compression']:g}": p["gather_incl_transpose_nonzero_tflops"]
                                         for p in pts if p["best_route"] == "gathered"}}
    return out


TRAFFIC_PROFILE = os.path.join("profiles", "linear_tc_kernel_bert_base_T4096.md")
TRAFFIC_SOURCES = ("paper_2009_08065_b200/csrc/bsp_linear_tc.cu", "paper_2009_08065_b200/csrc/bsp_tc.cuh")


def profiled_traffic():
    """DRAM bytes (read + write) of the four GEMM launches as ncu counted them, from the `traffic-record` line of
    the kernel's profile summary, or None when the kernel's sources have changed since that capture (the line
    carries their SHA-256) or the record is missing."""
    import hashlib
    root = os.path.dirname(os.path.abspath(__file__))
    try:
        h = hashlib.sha256()
        for f in TRAFFIC_SOURCES:
            with open(os.path.join(root, f), "rb") as fh:
                h.update(fh.read())
        with open(os.path.join(root, TRAFFIC_PROFILE)) as fh:
            line = next(l for l in fh if l.startswith("traffic-record:"))
        rec = dict(kv.split("=", 1) for kv in line.split(":", 1)[1].split())
        if rec.get("sha256") != h.hexdigest():
            return None
        return {k: int(v) for k, v in rec.items() if k != "sha256"}
    except (OSError, StopIteration, ValueError):
        return None


def section_8d_bytes(tokens, spec, kept_weights):
    """Algorithmic bytes of one pruned linear: X once, the kept values and one index per kept group, Y once, the bias."""
    return (2 * tokens * spec.k_in + 2 * kept_weights + 4 * (kept_weights // spec.block)
            + 2 * tokens * spec.n_out + 2 * spec.n_out)


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
    n_lin = len(layer.lin)

    # warm-up outside any graph (first calls set function attributes and the status word)
    for _ in range(max(args.warmup, 3)):
        layer.step()
    layer.bsp.bsp_linear_status()
    flops = layer.nonzero_flops()
    step_flops = sum(flops)
    kept = [f // (2 * wl.tokens) for f in flops]

    # The step as a CUDA graph, bracketed by two event nodes: it gives `value`.  The same call sequence cut
    # after the weight-side call and after each GEMM gives n_lin more graphs (prefixes); the difference between
    # two neighbouring prefixes is what a launch adds to the step, so the shares add up to the step exactly and
    # no event node sits between two kernels.  Every replay, of the step or of a prefix, follows its own L2 flush.
    ev = lambda: torch.cuda.Event(enable_timing=True, external=True)  # noqa: E731
    graphs = []
    for k in range(n_lin + 1):
        g, pair = torch.cuda.CUDAGraph(), (ev(), ev())
        with torch.cuda.graph(g):
            pair[0].record()
            layer.step(n_linears=k)
            pair[1].record()
        graphs.append((g, pair))
    graph, ev_step = graphs[n_lin]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    prefix_ms = [[] for _ in graphs]
    with ClockSampler(local_rank) as clocks:          # sampling starts with the warm-up replays: short runs still get samples
        for _ in range(max(args.warmup, 3)):
            for g, _pair in graphs:
                flush.zero_()
                g.replay()
        barrier()
        for _ in range(args.steps):
            for k in (n_lin, *range(n_lin)):          # the whole step first, then its prefixes
                g, pair = graphs[k]
                flush.zero_()                         # untimed: evict the inputs from L2
                g.replay()
                torch.cuda.synchronize()
                prefix_ms[k].append(pair[0].elapsed_time(pair[1]))
        barrier()
    layer.bsp.bsp_linear_status()
    total_ms = sum(prefix_ms[n_lin])

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

    def pipelined(n_steps, activations_only=False):
        ev_in = [torch.cuda.Event(), torch.cuda.Event()]
        ev_done = [torch.cuda.Event(), torch.cuda.Event()]
        ev_out = [torch.cuda.Event(), torch.cuda.Event()]
        for it in range(n_steps):
            k = it & 1
            lay, gr = sets[k]
            with torch.cuda.stream(s_in):
                if it >= 2:
                    s_in.wait_event(ev_done[k])        # the kernels of step it-2 have read this set's inputs
                lay.upload_inputs(activations_only)
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

    e2e_totals = []
    for act_only in (False, True):
        pipelined(max(args.warmup, 3), act_only)
        barrier()
        e_s.record()
        pipelined(args.steps, act_only)
        e_e.record()
        torch.cuda.synchronize()
        e2e_totals.append(e_s.elapsed_time(e_e))
        barrier()
    e2e_total_ms, e2e_act_total_ms = e2e_totals
    layer_b.bsp.bsp_linear_status()

    reduced = reduce_max([total_ms, e2e_total_ms, e2e_serial_total_ms, e2e_act_total_ms], device, world)
    total_ms, e2e_total_ms, e2e_serial_total_ms, e2e_act_total_ms = reduced

    if rank == 0:
        peaks, peak_src = measured_peaks()
        peak, hbm_peak = float(peaks["bf16_tflops"]), float(peaks["hbm_gbs"])
        value = job_throughput(world, step_flops, args.steps, total_ms)
        step_mean = statistics.mean(prefix_ms[n_lin])
        pre = [statistics.mean(v) for v in prefix_ms]                 # pre[k]: weight side + the first k GEMMs
        weight_ms = pre[0]
        share = [(pre[k + 1] if k + 1 < n_lin else step_mean) - pre[k] for k in range(n_lin)]
        gemm_total = sum(share)                                       # = step - weight side, by construction
        alg_bytes = [section_8d_bytes(wl.tokens, e["spec"], kept[i]) for i, e in enumerate(layer.lin)]
        t_tensor = step_flops / peak / 1e9                            # ms at the tensor peak
        t_hbm = sum(alg_bytes) / hbm_peak / 1e6                       # ms at the HBM peak, on the method's bytes
        hbm_binds = t_hbm >= t_tensor
        ach_tf, ach_gbs = step_flops / gemm_total / 1e9, sum(alg_bytes) / gemm_total / 1e6
        names = [e["spec"].name.split(".")[1] for e in layer.lin]
        traffic = profiled_traffic()
        if traffic is not None and sorted(traffic) != sorted(names):
            traffic = None
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(total_ms / args.steps, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": wl.name + " (one BERT-base encoder layer: QKV, attn-out, FFN-up+GELU, FFN-down; "
                            "tokens per GPU 4096; 16-row blocks; 3.0x compression)",
                "step": "bsp_prepare_batched (norms+gamma+penalty, keep flags, pack of the 4 matrices, in-place mode: a clearing "
                        "kernel and one kernel that reads W once) then the 4 GEMMs in sequence (bsp_linear_planned_ex on the "
                        "zero-expanded weights; the single chained launch bsp_linear_chain measured 6 % slower on this "
                        "workload); one CUDA graph",
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
                           "kernels of the neighbouring steps; every step copies all its inputs (activations, weights, "
                           "biases) in and its result out",
                    "one_step_at_a_time": round(job_throughput(world, step_flops, len(e2e_ms), e2e_serial_total_ms), 3),
                    "activations_only": {
                        "value": round(job_throughput(world, step_flops, args.steps, e2e_act_total_ms), 3),
                        "h2d_bytes_per_step": layer.h2d_bytes(True),
                        "how": "the same, with the weights and biases left on the device (they are 14.2 of the 20.5 MB)"}},
            "gpu_launches": args.steps * sum(layer.weight_side_launches + k for k in range(n_lin + 1)),
            "clocks": clocks.summary(),
            "roofline": {
                "kernel": "linear_tc_kernel (bsp_linear_planned_ex), the four launches of a step",
                "bound": "hbm" if hbm_binds else "tensor",
                "achieved": round(ach_gbs if hbm_binds else ach_tf, 2),
                "peak": hbm_peak if hbm_binds else peak, "unit": "GB/s" if hbm_binds else "TFLOP/s",
                "frac": round((ach_gbs / hbm_peak) if hbm_binds else (ach_tf / peak), 4),
                "binding": f"at this size the algorithmic bytes need {1e3 * t_hbm:.1f} us at the HBM peak and the non-zero FLOPs "
                           f"{1e3 * t_tensor:.1f} us at the bf16 peak: the {'HBM' if hbm_binds else 'tensor'} roofline is the one that binds",
                "tensor": {"achieved": round(ach_tf, 2), "peak": peak, "unit": "TFLOP/s", "frac": round(ach_tf / peak, 4),
                           "executed_tflops": round(sum(2 * wl.tokens * e["spec"].n_out * e["spec"].k_in for e in layer.lin) / gemm_total / 1e9, 1),
                           "note": "non-zero FLOPs; the kernel multiplies the zero-expanded weights, so it executes 3.0x as many"},
                "hbm": {"achieved": round(ach_gbs, 1), "peak": hbm_peak, "unit": "GB/s", "frac": round(ach_gbs / hbm_peak, 4)},
                "ms": round(gemm_total, 5),
                "how": "step minus the weight-side prefix; each launch's share = difference of two neighbouring prefixes of the "
                       "step, every prefix its own CUDA graph replayed after an L2 flush in the timed loop",
                "algorithmic_bytes": sum(alg_bytes),
                "algorithmic_bytes_formula": "per linear 2TK + 2 kept + 4 kept/d + 2TN + 2N (X once, kept values, one index per kept group, Y once, bias)",
                "traffic": sum(traffic.values()) if traffic else None,
                "traffic_per_launch": traffic,
                "traffic_note": "dram__bytes_read.sum + dram__bytes_write.sum of the four launches, one ncu capture per launch of "
                                "`bench.py --case <linear>` (" + TRAFFIC_PROFILE + "); not re-measured by this run, and null when the "
                                "kernel's sources no longer match the hash recorded with that capture",
                "peak_source": f"{'hbm_gbs' if hbm_binds else 'bf16_tflops burst'}, {peak_src}",
                "weight_side_ms": round(weight_ms, 5),
                "per_launch": {names[i]: {"ms": round(share[i], 5), "nonzero_tflops": round(flops[i] / share[i] / 1e9, 1),
                                          "algorithmic_gbs": round(alg_bytes[i] / share[i] / 1e6, 1)}
                               for i in range(n_lin)},
                "sum_check": {"weight_side_plus_launches_ms": round(weight_ms + gemm_total, 5), "step_ms": round(step_mean, 5)},
            },
        }
        if world == 1:
            line["weight_side_hbm"] = weight_side_bandwidth(device, peaks)
            line["retrain_step_hbm"] = retrain_step_bandwidth(device, peaks)
            line["dense_gemm_context"] = dense_context(wl, device)
            if not args.no_extras:
                line["other_workloads"] = other_workloads(device, peaks, args)
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
    """The BERT-large grid, one JSON line per point (see bert_large_grid)."""
    import torch
    torch.cuda.set_device(0)
    peaks, _ = measured_peaks()
    shapes = args.sweep_shapes.split(",") if args.sweep_shapes else None
    bert_large_grid(torch.device("cuda", 0), peaks, args.sweep_tokens, max(3, min(args.steps, 20)), shapes,
                    emit=lambda p: print(json.dumps({"sweep": "bert_large", **p}), flush=True))


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
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the figures of the other workloads (72-matrix stack, DistilBERT-shaped stack, BERT-large grid)")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    else:
        run_cuda(args)


def _rank_main(local_rank, args, port):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(args.gpus),
                      RANK=str(local_rank), LOCAL_RANK=str(local_rank))
    run_cuda(args)


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start the N ranks here, one per GPU (NCCL is only used for
    the barrier and the max-over-ranks of the times)."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_rank_main, args=(args, port), nprocs=args.gpus, join=True)


if __name__ == "__main__":
    main()
