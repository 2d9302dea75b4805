#!/usr/bin/env python
"""Benchmark of the MoE hot path (route -> histogram -> plan -> dispatch -> expert_ffn -> combine).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of the workload.  Prints ONE JSON line.
With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs the same workload
on its own batch: batches are independent, so there is no data-path collective ("weak" scaling);
the only communication is the barrier and the max-over-ranks of the elapsed time.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
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

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_07366_b200 import workloads as wl  # noqa: E402

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------- our arm
def run_ours(args):
    from paper_2506_07366_b200 import binding
    from paper_2506_07366_b200.layer import MoeLayer

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")

    w = wl.WORKLOADS[args.workload]
    A = 128
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, A)
    # every rank draws its own batch (same weights: data parallel replicas of the layer)
    wr, bias = wl.router(w, dev)
    w1, w3, w2 = wl.expert_weights(w, dev)
    x = wl.activations(w.scaled(number=w.number + 50 * rank), dev)
    layer = MoeLayer(shape, wr, bias, w1, w3, w2, device=local_rank)
    ctx = layer.ctx

    # the workload's stand-in for the predictor: computed once, outside the timed region, with the
    # library's own route + histogram (the prediction is an INPUT of the path)
    ctx.route(x, wr, bias, layer.topk_idx, layer.topk_w)
    ctx.histogram(layer.topk_idx, layer.hist)
    true_hist = layer.hist.cpu()
    if w.prediction == "true":
        pred = true_hist.clone()
    elif w.prediction == "noisy":
        pred = wl.noisy_prediction(w, true_hist)
    else:
        xprev = wl.activations(w, dev, previous=True)
        ctx.route(xprev, wr, bias, layer.topk_idx, layer.topk_w)
        ctx.histogram(layer.topk_idx, layer.hist)
        pred = layer.hist.cpu().clone()
    pred_dev = pred.to(dev, torch.int32)

    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    gemm_marks = []

    def step(record: bool):
        ctx.plan(pred_dev, w.S, layer.replicas, layer.slot_off, layer.slot_expert, layer.bound)
        ctx.route(x, wr, bias, layer.topk_idx, layer.topk_w)
        ctx.histogram(layer.topk_idx, layer.hist)
        ctx.dispatch(x, layer.topk_idx, layer.hist, layer.replicas, layer.slot_off, layer.slot_row_off,
                     layer.row_pair, layer.pair_row, layer.xp, layer.workspace)
        if record:
            a, b, c = ev(), ev(), ev()
            a.record(stream)
        ctx.expert_ffn_gate_up(layer.xp, layer.slot_row_off, layer.slot_expert, w1, w3, layer.h_ws)
        if record:
            b.record(stream)
        ctx.expert_ffn_down(layer.h_ws, layer.slot_row_off, layer.slot_expert, w2, layer.yp)
        if record:
            c.record(stream)
            gemm_marks.append((a, b, c))
        ctx.combine(layer.yp, layer.pair_row, layer.topk_w, layer.out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    ctx.check_status()

    sampler = ClockSampler(visible_gpu_index(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = ctx.launch_count()
    barrier()
    t0, t1 = ev(), ev()
    t0.record(stream)
    for _ in range(args.steps):
        step(True)
    t1.record(stream)
    barrier()
    elapsed_ms = t0.elapsed_time(t1)
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ctx.check_status()
    if dist is not None:
        tmax = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        elapsed_ms = float(tmax.item())
    value = world * w.T * args.steps / (elapsed_ms * 1e-3)

    gate_up_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in gemm_marks)
    down_ms = statistics.mean(b.elapsed_time(c) for _, b, c in gemm_marks)

    # end to end through the public layer API with host buffers (pinned), copies inside the timing
    xh = x.cpu().pin_memory()
    oh = torch.empty(w.T, w.D, dtype=torch.bfloat16).pin_memory()
    layer.plan(pred_dev)
    for _ in range(max(1, min(3, args.warmup))):
        layer.forward_host(xh, oh)
    barrier()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for _ in range(args.steps):
        layer.plan(pred_dev)
        layer.forward_host(xh, oh)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if dist is not None:
        tmax = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        e2e_ms = float(tmax.item())
    ctx.check_status()
    e2e_value = world * w.T * args.steps / (e2e_ms * 1e-3)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    flops_gate_up = 4.0 * w.R * w.D * w.F          # two of the three SwiGLU GEMMs, 2*R*D*F each
    achieved = flops_gate_up / (gate_up_ms * 1e-3) / 1e12
    ffn_tflops = 6.0 * w.R * w.D * w.F / ((gate_up_ms + down_ms) * 1e-3) / 1e12
    hist_np = true_hist.numpy().astype("float64")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S,
                   "row_align": A, "tokens_per_gpu": w.T, "prediction": w.prediction,
                   "skewness": float(hist_np.max() / (hist_np.sum() / w.E)),
                   "l2": "inputs larger than L2: %.2f GB of expert weights stream through it every step"
                         % (3 * w.E * w.D * w.F * 2 / 1e9)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": w.T * w.D * 2,
                "d2h_bytes_per_step": w.T * w.D * 2, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"kernel": "grouped_gemm_kernel<SwiGLU> (expert_ffn gate+up)", "bound": "tensor",
                     "achieved": achieved, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                     "frac": achieved / peaks["bf16_sustained"], "frac_of_burst_peak": achieved / peaks["bf16_burst"],
                     "peak_source": peaks["source"] + " (sustained bf16, kernel timed inside the step)",
                     "ms_per_launch": gate_up_ms, "traffic": None},
        "expert_ffn": {"tflops": ffn_tflops, "gate_up_ms": gate_up_ms, "down_ms": down_ms,
                       "frac_of_sustained_peak": ffn_tflops / peaks["bf16_sustained"]},
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, x, wr, bias, w1, w3, w2, pred)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------- oracle arm
def oracle_sample_step(w, xb, wrb, bias, w1, w3, w2, pred, n_tokens):
    """One pass of the oracle over the first n_tokens tokens of the batch."""
    import oracle
    sub = xb[:n_tokens]
    return oracle.moe_layer(sub, wrb, bias, w1, w3, w2, pred, K=w.K, S=w.S, gate_mode=w.gate_mode, row_align=1)


class _HostExperts:
    def __init__(self, t):
        self.t = t
        self.shape = tuple(t.shape)

    def __getitem__(self, e):
        return wl.bf16_bits(self.t[int(e)])


def cpu_baseline(w, x, wr, bias, w1, w3, w2, pred, n_tokens=None, seconds_hint=15.0):
    """Times the oracle, as it stands, on the host cores over a bounded sample of the workload."""
    import numpy as np
    from threadpoolctl import threadpool_info
    # the oracle's cost is dominated by 6*D*F MACs per routed pair at a few GFLOP/s per core
    if n_tokens is None:
        per_token = 6.0 * w.K * w.D * w.F
        n_tokens = int(max(8, min(w.T, seconds_hint * 2e10 / per_token)))
    xb, wrb, b = wl.bf16_bits(x[:n_tokens]), wl.bf16_bits(wr), bias.cpu().numpy()
    ex1, ex3, ex2 = _HostExperts(w1), _HostExperts(w3), _HostExperts(w2)
    t0 = time.perf_counter()
    oracle_sample_step(w, xb, wrb, b, ex1, ex3, ex2, np.asarray(pred), n_tokens)
    dt = time.perf_counter() - t0
    threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    return {"value": n_tokens / dt, "unit": UNIT, "cores": int(threads), "kind": "oracle",
            "sample": f"first {n_tokens} of {w.T} tokens of '{w.name}', all experts' weights, one pass "
                      f"(includes fetching each used expert's weights to the host), {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    w = wl.WORKLOADS[args.workload]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    wr, bias = wl.router(w, dev)
    w1, w3, w2 = wl.expert_weights(w, dev)
    x = wl.activations(w, dev)
    pred = np.full(w.E, w.R // w.E, dtype=np.int64)
    per_token = 6.0 * w.K * w.D * w.F
    n_tokens = int(max(8, min(w.T, 6.0 * 2e10 / per_token)))
    times = []
    for i in range(args.warmup + args.steps):
        r = cpu_baseline(w, x, wr, bias, w1, w3, w2, pred, n_tokens=n_tokens)
        if i >= args.warmup:
            times.append(n_tokens / r["value"])
    dt = sum(times)
    value = n_tokens * len(times) / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / len(times) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                             "sample": f"each step = first {n_tokens} of {w.T} tokens, all experts' weights"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="mixtral", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
