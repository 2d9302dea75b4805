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

# dram__bytes_read.sum + dram__bytes_write.sum of one gate+up GEMM launch, from the ncu captures
# summarised under profiles/ (bytes; None = not captured for the current kernel)
GATE_UP_DRAM_TRAFFIC = {"mixtral": 2064364288 + 241741568,          # profiles/ncu_traffic_mixtral.md
                        "fine_grained": 13879219968 + 228023552}    # profiles/ncu_traffic_fine_grained.md


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


# ------------------------------------------------------------------------------------- multi-rank plumbing
def rank_workload(w, rank: int):
    """The workload whose activations rank `rank` draws: same shapes and recipe, its own seed, so
    that every rank processes a different batch (data-parallel replicas, no data-path collective)."""
    return w.scaled(number=w.number + 50 * rank)


def max_over_ranks(ms: float, dist, device) -> float:
    """The job is as slow as its slowest rank."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, tokens_per_rank: int, steps: int, elapsed_ms: float) -> float:
    """Tokens per second over all ranks (weak scaling: every rank processes tokens_per_rank per step)."""
    return world * tokens_per_rank * steps / (elapsed_ms * 1e-3)


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
    x = wl.activations(rank_workload(w, rank), dev)
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
        ctx.route_histogram(x, wr, bias, layer.topk_idx, layer.topk_w, layer.hist)   # route + histogram fused
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
    elapsed_ms = max_over_ranks(elapsed_ms, dist, dev)
    value = whole_job_rate(world, w.T, args.steps, elapsed_ms)

    gate_up_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in gemm_marks)
    down_ms = statistics.mean(b.elapsed_time(c) for _, b, c in gemm_marks)

    # end to end through the public layer API with host buffers (pinned), copies inside the timing
    # (every step copies its batch in and its result out; HostPipeline overlaps the copies of
    # neighbouring steps with the compute, as a serving loop would)
    from paper_2506_07366_b200.layer import HostPipeline
    xh = [x.cpu().pin_memory() for _ in range(2)]
    oh = [torch.empty(w.T, w.D, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    pipe = HostPipeline(layer, depth=2)
    layer.plan(pred_dev)
    for i in range(max(2, min(3, args.warmup))):
        pipe.submit(xh[i % 2], oh[i % 2])
    pipe.drain()
    barrier()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for i in range(args.steps):
        layer.plan(pred_dev)
        pipe.submit(xh[i % 2], oh[i % 2])
    pipe.drain()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    ctx.check_status()
    e2e_value = whole_job_rate(world, w.T, args.steps, e2e_ms)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    kernels = per_call_timings(ctx, layer, w, x, wr, bias, w1, w3, w2, pred_dev, peaks) if world == 1 else None
    flops_gate_up = 4.0 * w.R * w.D * w.F          # two of the three SwiGLU GEMMs, 2*R*D*F each
    achieved = flops_gate_up / (gate_up_ms * 1e-3) / 1e12
    ffn_tflops = 6.0 * w.R * w.D * w.F / ((gate_up_ms + down_ms) * 1e-3) / 1e12
    hist_np = true_hist.numpy().astype("float64")
    active = int((hist_np > 0).sum())
    # slot loads of the last step: rows that carry a pair, counted per slot
    occupied = (layer.row_pair >= 0).to(torch.int64).cumsum(0)
    ends = layer.slot_row_off[1:].long().clamp(max=shape.Rcap) - 1
    starts = layer.slot_row_off[:-1].long() - 1
    cum_at = lambda i: torch.where(i >= 0, occupied[i.clamp(min=0)], torch.zeros_like(i))  # noqa: E731
    slot_loads = (cum_at(ends) - cum_at(starts)).cpu().numpy()
    err_dev = torch.zeros(1, dtype=torch.float64, device=dev)
    ctx.error_rate(pred_dev, layer.hist, err_dev)
    # a timed region of a few hundred ms runs at boost clocks: the burst peak is the fair denominator;
    # from a couple of seconds on, the power cap has settled and the sustained peak applies
    if elapsed_ms >= 2000.0:
        peak, peak_kind = peaks["bf16_sustained"], " (sustained bf16 GEMM: timed region >= 2 s)"
    else:
        peak, peak_kind = peaks["bf16_burst"], " (burst bf16 GEMM: timed region < 2 s, boost clocks)"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S,
                   "row_align": A, "tokens_per_gpu": w.T, "prediction": w.prediction,
                   "skewness": float(hist_np.max() / (hist_np.sum() / w.E)),
                   # the paper's load statistics of this batch, from the library's own outputs: the
                   # bottleneck slot's load over the even share after duplication, the planner's
                   # predicted bound, and the error rate of the prediction that drove the plan
                   "skewness_after_plan": float(slot_loads.max() / (w.R / w.S)),
                   "max_slot_load": int(slot_loads.max()), "plan_bound": int(layer.bound.item()),
                   "prediction_error_rate": float(err_dev.item()),
                   "l2": "inputs larger than L2: %.2f GB of expert weights stream through it every step"
                         % (3 * w.E * w.D * w.F * 2 / 1e9)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": w.T * w.D * 2,
                "d2h_bytes_per_step": w.T * w.D * 2, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"kernel": "grouped_gemm_kernel<SwiGLU> (expert_ffn gate+up)", "bound": "tensor",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "frac_of_burst_peak": achieved / peaks["bf16_burst"],
                     "frac_of_sustained_peak": achieved / peaks["bf16_sustained"],
                     "peak_source": peaks["source"] + peak_kind,
                     "ms_per_launch": gate_up_ms, "traffic": GATE_UP_DRAM_TRAFFIC.get(w.name)},
        "expert_ffn": {"tflops": ffn_tflops, "gate_up_ms": gate_up_ms, "down_ms": down_ms,
                       "frac_of_sustained_peak": ffn_tflops / peaks["bf16_sustained"],
                       # the other roof of the grouped GEMMs: every expert that received tokens has its
                       # weights streamed from HBM once per GEMM (binding when slots hold few rows)
                       "active_experts": active,
                       "gate_up_weight_gbs": active * 2.0 * w.D * w.F * 2 / (gate_up_ms * 1e-3) / 1e9,
                       "down_weight_gbs": active * 1.0 * w.D * w.F * 2 / (down_ms * 1e-3) / 1e9,
                       "gate_up_weight_frac_of_hbm_peak":
                           active * 2.0 * w.D * w.F * 2 / (gate_up_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
    }
    if kernels is not None:
        line["calls_cold_l2"] = kernels
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, x, wr, bias, w1, w3, w2, pred)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def per_call_timings(ctx, layer, w, x, wr, bias, w1, w3, w2, pred_dev, peaks, iters=7):
    """Each library call timed alone (CUDA events on the launching stream, median of `iters`) with L2
    flushed before every call by overwriting a 512 MB buffer, against the call's algorithmic HBM bytes
    or flops.  The interval between the two events also holds the stream's launch gaps and the event
    records themselves (`event_pair` = the same measurement with nothing in between), which matters
    for calls of a few microseconds; kernel-only durations are in the ncu launch lists.  These
    numbers explain the step time; they are not part of the timed step."""
    stream = torch.cuda.current_stream()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=x.device)
    R, T, D, F, E, K = w.R, w.T, w.D, w.F, w.E, w.K
    ctx.plan(pred_dev, w.S, layer.replicas, layer.slot_off, layer.slot_expert, layer.bound)
    calls = [
        ("plan", lambda: ctx.plan(pred_dev, w.S, layer.replicas, layer.slot_off, layer.slot_expert, layer.bound),
         None, None),
        ("route", lambda: ctx.route(x, wr, bias, layer.topk_idx, layer.topk_w),
         2.0 * T * D + 2.0 * E * D + 8.0 * T * K, 2.0 * T * D * E),
        ("histogram", lambda: ctx.histogram(layer.topk_idx, layer.hist), 4.0 * R, None),
        ("route_histogram", lambda: ctx.route_histogram(x, wr, bias, layer.topk_idx, layer.topk_w, layer.hist),
         2.0 * T * D + 2.0 * E * D + 8.0 * T * K, 2.0 * T * D * E),
        ("dispatch", lambda: ctx.dispatch(x, layer.topk_idx, layer.hist, layer.replicas, layer.slot_off,
                                          layer.slot_row_off, layer.row_pair, layer.pair_row, layer.xp,
                                          layer.workspace), 2.0 * T * D + 2.0 * R * D + 12.0 * R, None),
        ("expert_ffn_gate_up", lambda: ctx.expert_ffn_gate_up(layer.xp, layer.slot_row_off, layer.slot_expert, w1, w3,
                                                              layer.h_ws), None, 4.0 * R * D * F),
        ("expert_ffn_down", lambda: ctx.expert_ffn_down(layer.h_ws, layer.slot_row_off, layer.slot_expert, w2,
                                                        layer.yp), None, 2.0 * R * D * F),
        ("combine", lambda: ctx.combine(layer.yp, layer.pair_row, layer.topk_w, layer.out),
         2.0 * R * D + 2.0 * T * D + 8.0 * R, None),
    ]
    out = {}
    calls.append(("event_pair", lambda: None, None, None))
    for name, fn, nbytes, flops in calls:
        times = []
        for _ in range(iters):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            b.synchronize()
            times.append(a.elapsed_time(b))
        ms = statistics.median(times)
        rec = {"us": ms * 1e3}
        if nbytes is not None:
            rec["gbs"] = nbytes / (ms * 1e-3) / 1e9
            rec["frac_of_hbm_peak"] = rec["gbs"] / peaks["hbm_gbs"]
        if flops is not None and name.startswith("expert"):
            rec["tflops"] = flops / (ms * 1e-3) / 1e12
            rec["frac_of_burst_peak"] = rec["tflops"] / peaks["bf16_burst"]
        out[name] = rec
    ctx.check_status()
    return out


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


def cpu_baseline(w, x, wr, bias, w1, w3, w2, pred, n_tokens=None, seconds_hint=120.0):
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
