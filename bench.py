#!/usr/bin/env python
"""Benchmark of the MoE hot path (plan -> route + histogram -> dispatch -> expert_ffn -> combine).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of the workload.  Prints ONE JSON line.
The default workload is `mixtral_skew` (Mixtral-8x7B layer shape, 16384 tokens, heavy routing skew,
16 slots for 8 experts, noisy predicted histogram): the largest single-GPU configuration, and one in
which the duplication plan really replicates experts inside the timed step.  The other full-size
workloads are measured after it in the same process and reported in the `per_workload` block.
With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs the same workload
on its own batch: batches are independent, so there is no data-path collective ("weak" scaling);
the only communication is the barrier and the max-over-ranks of the elapsed time.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
`--record-traffic CSV` (no GPU needed) turns an `ncu --csv` capture of the DRAM byte counters into
profiles/dram_traffic.json, the file the `roofline.traffic` figure is read from.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
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
DEFAULT_WORKLOAD = "mixtral_skew"
OTHER_WORKLOADS = ("mixtral", "many_expert", "fine_grained")
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "dram_traffic.json")
GEMM_SOURCES = ("expert_ffn.cu", "sm100.cuh")       # what the captured DRAM traffic depends on


# ------------------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def gemm_source_hash() -> str:
    h = hashlib.sha256()
    for name in GEMM_SOURCES:
        with open(os.path.join(ROOT, "paper_2506_07366_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, pairs: int):
    """dram__bytes_read.sum + dram__bytes_write.sum of one gate+up GEMM launch of `workload`, from
    the ncu capture recorded in profiles/dram_traffic.json; None when there is no capture or the
    kernel's sources have changed since it was taken.  A capture of a reduced cut of the workload
    (fewer routed pairs, same layer) is scaled to a full launch by the pairs processed."""
    try:
        with open(TRAFFIC_JSON) as f:
            rec = json.load(f)["gate_up"][workload]
    except (OSError, KeyError, ValueError):
        return None
    if rec.get("source_hash") != gemm_source_hash():
        return None
    return (rec["dram_read_bytes"] + rec["dram_write_bytes"]) * (pairs / rec["pairs_in_capture"])


def record_traffic(csv_path: str, workload: str, pairs: int):
    """Reads an `ncu --csv` log that holds dram__bytes_read.sum / dram__bytes_write.sum of
    grouped_gemm_kernel launches and stores the per-launch mean of the gate+up and the down GEMM."""
    rows = []
    with open(csv_path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    for r in csv.DictReader(lines):
        rows.append(r)
    out = {}
    for key, tag in (("gate_up", "grouped_gemm_kernel<1,"), ("down", "grouped_gemm_kernel<0,")):
        acc = {"dram__bytes_read.sum": [], "dram__bytes_write.sum": []}
        for r in rows:
            if tag not in r.get("Kernel Name", ""):
                continue
            m = r.get("Metric Name")
            if m in acc:
                v = float(r["Metric Value"].replace(",", ""))
                unit = r.get("Metric Unit", "byte").lower()
                v *= {"byte": 1.0, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9}.get(unit, 1.0)
                acc[m].append(v)
        if acc["dram__bytes_read.sum"]:
            out[key] = {"dram_read_bytes": statistics.mean(acc["dram__bytes_read.sum"]),
                        "dram_write_bytes": statistics.mean(acc["dram__bytes_write.sum"]),
                        "launches": len(acc["dram__bytes_read.sum"]), "pairs_in_capture": pairs,
                        "source_hash": gemm_source_hash()}
    if not out:
        raise SystemExit(f"{csv_path}: no grouped_gemm_kernel DRAM counters found")
    data = {}
    if os.path.exists(TRAFFIC_JSON):
        with open(TRAFFIC_JSON) as f:
            data = json.load(f)
    for key, rec in out.items():
        data.setdefault(key, {})[workload] = rec
    with open(TRAFFIC_JSON, "w") as f:
        json.dump(data, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(out))


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
class Bench:
    """One workload resident on the device: layer, inputs, prediction."""

    def __init__(self, w, rank: int, local_rank: int):
        from paper_2506_07366_b200 import binding
        from paper_2506_07366_b200.layer import MoeLayer, ROW_ALIGN
        self.A = ROW_ALIGN
        self.w, self.dev = w, torch.device("cuda", local_rank)
        dev = self.dev
        self.shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, self.A)
        # every rank draws its own batch (same weights: data parallel replicas of the layer)
        self.wr, self.bias = wl.router(w, dev)
        self.w1, self.w3, self.w2 = wl.expert_weights(w, dev)
        self.x = wl.activations(rank_workload(w, rank), dev)
        self.layer = layer = MoeLayer(self.shape, self.wr, self.bias, self.w1, self.w3, self.w2, device=local_rank)
        self.ctx = ctx = layer.ctx
        # the workload's stand-in for the predictor: computed once, outside the timed region, with the
        # library's own route + histogram (the prediction is an INPUT of the path)
        ctx.route(self.x, self.wr, self.bias, layer.topk_idx, layer.topk_w)
        ctx.histogram(layer.topk_idx, layer.hist)
        self.true_hist = layer.hist.cpu()
        if w.prediction == "true":
            pred = self.true_hist.clone()
        elif w.prediction == "noisy":
            pred = wl.noisy_prediction(w, self.true_hist)
        else:
            xprev = wl.activations(w, dev, previous=True)
            ctx.route(xprev, self.wr, self.bias, layer.topk_idx, layer.topk_w)
            ctx.histogram(layer.topk_idx, layer.hist)
            pred = layer.hist.cpu().clone()
        self.pred = pred
        self.pred_dev = pred.to(dev, torch.int32)
        self.gemm_marks = []

    def step(self, record: bool):
        L, c, w = self.layer, self.ctx, self.w
        c.plan(self.pred_dev, w.S, L.replicas, L.slot_off, L.slot_expert, L.bound)
        # route + histogram + the counts dispatch ranks with in one kernel, dispatch in one
        c.route_prepare(self.x, self.wr, self.bias, L.topk_idx, L.topk_w, L.hist, L.workspace)
        c.dispatch_prepared(self.x, L.topk_idx, L.hist, L.replicas, L.slot_off, L.slot_row_off, L.row_pair,
                            L.pair_row, L.xp, L.workspace)
        stream = torch.cuda.current_stream()
        if record:
            a, b, e = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record(stream)
        c.expert_ffn_gate_up(L.xp, L.slot_row_off, L.slot_expert, self.w1, self.w3, L.h_ws)
        if record:
            b.record(stream)
        c.expert_ffn_down(L.h_ws, L.slot_row_off, L.slot_expert, self.w2, L.yp)
        if record:
            e.record(stream)
            self.gemm_marks.append((a, b, e))
        c.combine(L.yp, L.pair_row, L.topk_w, L.out)

    def timed_steps(self, steps: int, warmup: int, barrier):
        """W warm-up steps, then exactly `steps` steps between two events on the launching stream."""
        stream = torch.cuda.current_stream()
        for _ in range(warmup):
            self.step(False)
        barrier()
        self.ctx.check_status()
        self.gemm_marks = []
        launches0 = self.ctx.launch_count()
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            self.step(True)
        t1.record(stream)
        barrier()
        self.ctx.check_status()
        ms = t0.elapsed_time(t1)
        gate_up = statistics.mean(a.elapsed_time(b) for a, b, _ in self.gemm_marks)
        down = statistics.mean(b.elapsed_time(e) for _, b, e in self.gemm_marks)
        return ms, gate_up, down, self.ctx.launch_count() - launches0

    def e2e_steps(self, steps: int, warmup: int, barrier):
        """End to end through the public layer API with pinned host buffers, copies inside the timing
        (every step copies its batch in and its result out; HostPipeline overlaps the copies of
        neighbouring steps with the compute, as a serving loop would)."""
        from paper_2506_07366_b200.layer import HostPipeline
        w, layer = self.w, self.layer
        stream = torch.cuda.current_stream()
        xh = [self.x.cpu().pin_memory() for _ in range(2)]
        oh = [torch.empty(w.T, w.D, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        pipe = HostPipeline(layer, depth=2)
        layer.plan(self.pred_dev)
        for i in range(max(2, min(3, warmup))):
            pipe.submit(xh[i % 2], oh[i % 2])
        pipe.drain()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            layer.plan(self.pred_dev)
            pipe.submit(xh[i % 2], oh[i % 2])
        pipe.drain()
        e1.record(stream)
        barrier()
        self.ctx.check_status()
        return e0.elapsed_time(e1)

    def load_statistics(self) -> dict:
        """The paper's load statistics of the last batch, from the library's own outputs: skewness
        before and after duplication, the planner's bound, the prediction's error rate."""
        w, layer = self.w, self.layer
        hist = self.true_hist.numpy().astype("float64")
        occupied = (layer.row_pair >= 0).to(torch.int64).cumsum(0)
        ends = layer.slot_row_off[1:].long().clamp(max=self.shape.Rcap) - 1
        starts = layer.slot_row_off[:-1].long() - 1
        cum_at = lambda i: torch.where(i >= 0, occupied[i.clamp(min=0)], torch.zeros_like(i))  # noqa: E731
        slot_loads = (cum_at(ends) - cum_at(starts)).cpu().numpy()
        err_dev = torch.zeros(1, dtype=torch.float64, device=self.dev)
        self.ctx.error_rate(self.pred_dev, layer.hist, err_dev)
        return {"skewness": float(hist.max() / (hist.sum() / w.E)),
                "skewness_after_plan": float(slot_loads.max() / (w.R / w.S)),
                "max_slot_load": int(slot_loads.max()), "plan_bound": int(layer.bound.item()),
                "prediction_error_rate": float(err_dev.item()), "active_experts": int((hist > 0).sum()),
                "max_replicas": int(layer.replicas.max().item())}

    def per_call_timings(self, peaks, iters=7):
        """Each library call timed alone (CUDA events on the launching stream, median of `iters`) with
        a cold L2: before every call a 512 MB buffer is READ, which leaves L2 full of clean lines of
        that buffer, so the call's inputs come from HBM and its stores evict nothing dirty.  The
        interval between the two events also holds the launch latency of the stream and the event
        records themselves (`event_pair` = the same measurement with nothing in between; calls that
        launch two kernels pay the gap twice).  The loop starts after a one-second pause: right after
        a run of steps the chip is still at its power cap (SM clock near 1.4 GHz instead of 1.97) and
        these short latency-bound calls would read up to 1.5x longer.  These numbers explain the step
        time; they are not part of the timed step."""
        w, L, c = self.w, self.layer, self.ctx
        torch.cuda.synchronize()
        time.sleep(1.0)
        stream = torch.cuda.current_stream()
        evict = torch.zeros(128 << 20, dtype=torch.float32, device=self.dev)
        R, T, D, F, E, K = w.R, w.T, w.D, w.F, w.E, w.K
        c.plan(self.pred_dev, w.S, L.replicas, L.slot_off, L.slot_expert, L.bound)
        calls = [
            ("plan", lambda: c.plan(self.pred_dev, w.S, L.replicas, L.slot_off, L.slot_expert, L.bound), None, None),
            ("route", lambda: c.route(self.x, self.wr, self.bias, L.topk_idx, L.topk_w),
             2.0 * T * D + 2.0 * E * D + 8.0 * T * K, 2.0 * T * D * E),
            ("histogram", lambda: c.histogram(L.topk_idx, L.hist), 4.0 * R, None),
            ("route_histogram", lambda: c.route_histogram(self.x, self.wr, self.bias, L.topk_idx, L.topk_w, L.hist),
             2.0 * T * D + 2.0 * E * D + 8.0 * T * K, 2.0 * T * D * E),
            ("dispatch", lambda: c.dispatch(self.x, L.topk_idx, L.hist, L.replicas, L.slot_off, L.slot_row_off,
                                            L.row_pair, L.pair_row, L.xp, L.workspace),
             2.0 * T * D + 2.0 * R * D + 12.0 * R, None),
            ("route_prepare", lambda: c.route_prepare(self.x, self.wr, self.bias, L.topk_idx, L.topk_w, L.hist,
                                                      L.workspace),
             2.0 * T * D + 2.0 * E * D + 8.0 * T * K, 2.0 * T * D * E),
            ("dispatch_prepared", lambda: c.dispatch_prepared(self.x, L.topk_idx, L.hist, L.replicas, L.slot_off,
                                                              L.slot_row_off, L.row_pair, L.pair_row, L.xp,
                                                              L.workspace),
             2.0 * T * D + 2.0 * R * D + 12.0 * R, None),
            ("expert_ffn_gate_up", lambda: c.expert_ffn_gate_up(L.xp, L.slot_row_off, L.slot_expert, self.w1, self.w3,
                                                                L.h_ws), None, 4.0 * R * D * F),
            ("expert_ffn_down", lambda: c.expert_ffn_down(L.h_ws, L.slot_row_off, L.slot_expert, self.w2, L.yp),
             None, 2.0 * R * D * F),
            ("combine", lambda: c.combine(L.yp, L.pair_row, L.topk_w, L.out), 2.0 * R * D + 2.0 * T * D + 8.0 * R, None),
            ("event_pair", lambda: None, None, None),
        ]
        out = {}
        for name, fn, nbytes, flops in calls:
            times = []
            for _ in range(iters):
                evict.sum()
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
        c.check_status()
        return out

    def ffn_summary(self, gate_up_ms, down_ms, peaks, active) -> dict:
        w = self.w
        ffn_tflops = 6.0 * w.R * w.D * w.F / ((gate_up_ms + down_ms) * 1e-3) / 1e12
        # the other roof of the grouped GEMMs: every expert that received tokens has its weights
        # streamed from HBM once per GEMM, and the activations go in and out once (binding when
        # slots hold few rows)
        bytes_gate_up = active * 2.0 * w.D * w.F * 2 + 2.0 * w.R * w.D + 2.0 * w.R * w.F
        bytes_down = active * 1.0 * w.D * w.F * 2 + 2.0 * w.R * w.F + 2.0 * w.R * w.D
        return {"tflops": ffn_tflops, "gate_up_ms": gate_up_ms, "down_ms": down_ms,
                "frac_of_burst_peak": ffn_tflops / peaks["bf16_burst"],
                "frac_of_sustained_peak": ffn_tflops / peaks["bf16_sustained"],
                "gate_up_frac_of_burst_peak": 4.0 * w.R * w.D * w.F / (gate_up_ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                "down_frac_of_burst_peak": 2.0 * w.R * w.D * w.F / (down_ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                "gate_up_hbm_gbs": bytes_gate_up / (gate_up_ms * 1e-3) / 1e9,
                "down_hbm_gbs": bytes_down / (down_ms * 1e-3) / 1e9,
                "gate_up_frac_of_hbm_peak": bytes_gate_up / (gate_up_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "down_frac_of_hbm_peak": bytes_down / (down_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    def close(self):
        self.layer.ctx.close()


def compact_record(b: Bench, peaks, steps: int, barrier) -> dict:
    """The short form reported for the workloads other than the headline one."""
    ms, gate_up, down, _ = b.timed_steps(steps, 3, barrier)
    stats = b.load_statistics()
    calls = b.per_call_timings(peaks, iters=5)
    ffn = b.ffn_summary(gate_up, down, peaks, stats["active_experts"])
    w = b.w
    return {"T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S, "steps": steps,
            "ms_per_step": ms / steps, "tokens_per_s": w.T * steps / (ms * 1e-3),
            "ffn_tflops": ffn["tflops"], "gate_up_ms": gate_up, "down_ms": down,
            "gate_up_frac_of_burst_peak": ffn["gate_up_frac_of_burst_peak"],
            "down_frac_of_burst_peak": ffn["down_frac_of_burst_peak"],
            "gate_up_frac_of_hbm_peak": ffn["gate_up_frac_of_hbm_peak"],
            "down_frac_of_hbm_peak": ffn["down_frac_of_hbm_peak"],
            "cold_l2_us": {k: round(calls[k]["us"], 2)
                           for k in ("route_prepare", "dispatch_prepared", "combine", "plan")},
            "frac_of_hbm_peak": {k: round(calls[k]["frac_of_hbm_peak"], 3)
                                 for k in ("route_prepare", "dispatch_prepared", "combine")},
            "skewness": stats["skewness"], "skewness_after_plan": stats["skewness_after_plan"]}


def run_ours(args):
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

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.WORKLOADS[args.workload]
    b = Bench(w, rank, local_rank)
    sampler = ClockSampler(visible_gpu_index(local_rank))
    for _ in range(args.warmup):            # warm-up before the clock sampler starts, too
        b.step(False)
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    elapsed_ms, gate_up_ms, down_ms, launches = b.timed_steps(args.steps, 0, barrier)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = max_over_ranks(elapsed_ms, dist, dev)
    value = whole_job_rate(world, w.T, args.steps, elapsed_ms)
    e2e_ms = max_over_ranks(b.e2e_steps(args.steps, args.warmup, barrier), dist, dev)
    e2e_value = whole_job_rate(world, w.T, args.steps, e2e_ms)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    stats = b.load_statistics()
    calls = b.per_call_timings(peaks) if world == 1 else None
    ffn = b.ffn_summary(gate_up_ms, down_ms, peaks, stats["active_experts"])
    achieved = 4.0 * w.R * w.D * w.F / (gate_up_ms * 1e-3) / 1e12      # two of the three SwiGLU GEMMs, 2*R*D*F each
    # a timed region of a few hundred ms runs at boost clocks: the burst peak is the fair denominator;
    # from a couple of seconds on, the power cap has settled and the sustained peak applies
    if elapsed_ms >= 2000.0:
        peak, peak_kind = peaks["bf16_sustained"], " (sustained bf16 GEMM: timed region >= 2 s)"
    else:
        peak, peak_kind = peaks["bf16_burst"], " (burst bf16 GEMM: timed region < 2 s, boost clocks)"
    config = {"workload": w.name, "T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S,
              "row_align": b.A, "tokens_per_gpu": w.T, "prediction": w.prediction,
              "l2": "inputs larger than L2: %.2f GB of expert weights stream through it every step"
                    % (3 * w.E * w.D * w.F * 2 / 1e9)}
    config.update({k: stats[k] for k in ("skewness", "skewness_after_plan", "max_slot_load", "plan_bound",
                                         "prediction_error_rate", "max_replicas")})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": w.T * w.D * 2,
                "d2h_bytes_per_step": w.T * w.D * 2, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"kernel": "grouped_gemm_kernel<SwiGLU> (expert_ffn gate+up)", "bound": "tensor",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "frac_of_burst_peak": achieved / peaks["bf16_burst"],
                     "frac_of_sustained_peak": achieved / peaks["bf16_sustained"],
                     "peak_source": peaks["source"] + peak_kind,
                     "ms_per_launch": gate_up_ms, "traffic": recorded_traffic(w.name, w.R)},
        "expert_ffn": ffn,
    }
    if calls is not None:
        line["calls_cold_l2"] = calls
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, b.x, b.wr, b.bias, b.w1, b.w3, b.w2, b.pred)
    if world == 1 and not args.no_per_workload:
        per = {}
        b.close()
        del b
        for name in OTHER_WORKLOADS:
            if name == w.name:
                continue
            torch.cuda.empty_cache()
            try:                            # a failure here must not cost the headline measurement above
                ob = Bench(wl.WORKLOADS[name], 0, local_rank)
                per[name] = compact_record(ob, peaks, args.per_workload_steps, barrier)
                ob.close()
                del ob
            except Exception as exc:        # noqa: BLE001 - reported in the line instead
                per[name] = {"error": f"{type(exc).__name__}: {exc}"[:300]}
        line["per_workload"] = per
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------- oracle arm
class _HostExperts:
    """w[e] -> host bf16 bits of one expert's matrix, fetched from the device on first use."""

    def __init__(self, t):
        self.t, self.shape, self.cache = t, tuple(t.shape), {}

    def __getitem__(self, e):
        e = int(e)
        if e not in self.cache:
            self.cache[e] = wl.bf16_bits(self.t[e])
        return self.cache[e]


def oracle_sample_tokens(w) -> int:
    """Tokens per oracle pass: sized so that one pass takes a few seconds on the host cores (the
    cost is about 6*D*F fp64 multiply-adds per routed pair plus decoding every used expert's weights)."""
    per_token = 6.0 * w.K * w.D * w.F
    return int(max(8, min(w.T, 50.0 * 2e10 / per_token)))


class OracleSample:
    """The first n tokens of a workload's batch with everything the oracle needs on the host."""

    def __init__(self, w, x, wr, bias, w1, w3, w2, pred):
        import numpy as np
        self.w, self.n = w, oracle_sample_tokens(w)
        self.xb, self.wrb, self.b = wl.bf16_bits(x[:self.n]), wl.bf16_bits(wr), bias.cpu().numpy()
        self.experts = [_HostExperts(t) for t in (w1, w3, w2)]
        self.pred = np.asarray(pred)

    def one_pass(self) -> float:
        """One pass of the oracle, as it stands, over the sample; returns the seconds it took."""
        import oracle
        w = self.w
        t0 = time.perf_counter()
        oracle.moe_layer(self.xb, self.wrb, self.b, *self.experts, self.pred, K=w.K, S=w.S, gate_mode=w.gate_mode,
                         row_align=1)
        return time.perf_counter() - t0

    def describe(self) -> str:
        return (f"first {self.n} of {self.w.T} tokens of '{self.w.name}', all experts' weights (bf16 bits on the "
                f"host, fetched before the timing; decoding them to fp64 is part of every pass)")


def host_threads() -> int:
    from threadpoolctl import threadpool_info
    return int(max([p.get("num_threads", 1) for p in threadpool_info()] + [1]))


def cpu_baseline(w, x, wr, bias, w1, w3, w2, pred, passes=2):
    """Times the oracle, as it stands, on the host cores over a bounded sample of the workload: one
    untimed pass (it also brings the weights to the host), then `passes` timed ones."""
    s = OracleSample(w, x, wr, bias, w1, w3, w2, pred)
    s.one_pass()
    dt = sum(s.one_pass() for _ in range(passes))
    return {"value": s.n * passes / dt, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
            "sample": f"{s.describe()}; {passes} passes, {dt / passes:.1f} s each"}


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
    s = OracleSample(w, x, wr, bias, w1, w3, w2, pred)          # the same sample as the cpu_baseline leg
    for _ in range(max(1, args.warmup)):
        s.one_pass()
    times = [s.one_pass() for _ in range(args.steps)]
    dt = sum(times)
    value = s.n * len(times) / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / len(times) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "T": w.T, "D": w.D, "F": w.F, "E": w.E, "K": w.K, "S": w.S},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                             "sample": f"each step = {s.describe()}"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the short measurements of the other full-size workloads")
    ap.add_argument("--per-workload-steps", type=int, default=10)
    ap.add_argument("--record-traffic", metavar="NCU_CSV",
                    help="store the grouped GEMMs' DRAM byte counters of an ncu --csv log (taken on "
                         "--workload, --traffic-pairs routed pairs per launch) in profiles/dram_traffic.json")
    ap.add_argument("--traffic-pairs", type=int, default=0)
    args = ap.parse_args()
    if args.record_traffic:
        w = wl.WORKLOADS[args.workload]
        record_traffic(args.record_traffic, w.name, args.traffic_pairs or w.R)
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
