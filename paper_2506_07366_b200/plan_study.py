"""Plan-quality study: what expert duplication buys on a B200, measured.

The paper (Section 2) models the expert-parallel FFN latency of a layer as the even-share latency
multiplied by the skewness (the most loaded device sets the pace), and after prediction-driven
duplication by (1 + error) in its typical case (Section 3.3).  Here each logical slot stands for one
device of such a deployment, so the layer's FFN latency is the time the *most loaded slot* needs.
For one workload this script sweeps the number of extra replica slots and the noise of the predicted
histogram, lets the library route, count, plan and dispatch, reads the slot loads back, and times
the grouped SwiGLU FFN of a single slot holding (a) the even share R/S, (b) the largest slot load.
It prints, per setting: skewness before and after the plan, the planner's bound, the measured
bottleneck time, and its ratio to the even-share time next to the paper's model of that ratio.

  python -m paper_2506_07366_b200.plan_study [--workload mixtral_skew] [--extra 0 2 4 8 16] [--noise 0 0.1 0.3]

Everything on the device runs in libmoegps.so; this file only draws inputs, calls the library and
prints.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import workloads as wl
from .binding import Context, Shape, workspace_bytes


def _slot_ffn_ms(rows: int, w, w1, w3, w2, dev, cache, iters=5):
    """Median time (ms) of expert_ffn over one slot of `rows` rows of expert 0."""
    rows = max(1, int(rows))
    if rows in cache:
        return cache[rows]
    shape = Shape(rows, w.D, w.F, 1, 1, 1, 0, 128)
    ctx = Context(shape)
    xp = torch.randn(shape.Rcap, w.D, device=dev, dtype=torch.float32).to(torch.bfloat16)
    h = torch.empty(shape.Rcap, w.F, dtype=torch.bfloat16, device=dev)
    yp = torch.empty(shape.Rcap, w.D, dtype=torch.bfloat16, device=dev)
    sro = torch.tensor([0, rows], dtype=torch.int32, device=dev)
    sexp = torch.zeros(1, dtype=torch.int32, device=dev)
    a1, a3, a2 = w1[:1].contiguous(), w3[:1].contiguous(), w2[:1].contiguous()
    stream = torch.cuda.current_stream()
    times = []
    for i in range(iters + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.expert_ffn(xp, sro, sexp, a1, a3, a2, h, yp)
        e1.record(stream)
        e1.synchronize()
        if i >= 2:
            times.append(e0.elapsed_time(e1))
    ctx.check_status()
    cache[rows] = statistics.median(times)
    return cache[rows]


def study(name: str, extras, noises, device=0):
    torch.cuda.set_device(device)
    dev = torch.device("cuda", device)
    w = wl.WORKLOADS[name]
    wr, bias = wl.router(w, dev)
    x = wl.activations(w, dev)
    w1, w3, w2 = wl.expert_weights(w.scaled(E=1), dev)      # one expert's weights are enough
    i32 = dict(dtype=torch.int32, device=dev)
    # true routing of the batch (library route + histogram)
    base = Context(Shape(w.T, w.D, w.F, w.E, w.K, w.E, w.gate_mode, 1))
    topk_idx = torch.empty(w.T, w.K, **i32)
    topk_w = torch.empty(w.T, w.K, dtype=torch.float32, device=dev)
    hist = torch.empty(w.E, **i32)
    base.route_histogram(x, wr, bias, topk_idx, topk_w, hist)
    base.check_status()
    n = hist.cpu().to(torch.float64)
    R = w.R
    skew_before = float(n.max() / (R / w.E))
    cache = {}
    rows = []
    for extra in extras:
        S = w.E + extra
        shape = Shape(w.T, w.D, w.F, w.E, w.K, S, w.gate_mode, 1)    # row_align 1: offsets = exact loads
        ctx = Context(shape)
        replicas, slot_off = torch.empty(w.E, **i32), torch.empty(w.E + 1, **i32)
        slot_expert, bound = torch.empty(S, **i32), torch.empty(1, **i32)
        slot_row_off, row_pair = torch.empty(S + 1, **i32), torch.empty(shape.Rcap, **i32)
        pair_row = torch.empty(w.T, w.K, **i32)
        xp = torch.empty(shape.Rcap, w.D, dtype=torch.bfloat16, device=dev)
        ws = torch.empty(max(16, workspace_bytes(shape)), dtype=torch.uint8, device=dev)
        err = torch.zeros(1, dtype=torch.float64, device=dev)
        for sigma in noises:
            g = torch.Generator(device="cpu")
            g.manual_seed(w.seed + 6 + int(1000 * sigma))
            z = torch.randn(w.E, generator=g, dtype=torch.float64)
            pred = torch.clamp(torch.round(n * (1.0 + sigma * z)), min=0).to(torch.int32).to(dev)
            ctx.plan(pred, S, replicas, slot_off, slot_expert, bound)
            ctx.dispatch(x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp, ws)
            ctx.error_rate(pred, hist, err)
            ctx.check_status()
            loads = (slot_row_off[1:] - slot_row_off[:-1]).cpu()
            max_load, even = int(loads.max()), -(-R // S)
            t_max = _slot_ffn_ms(max_load, w, w1, w3, w2, dev, cache)
            t_even = _slot_ffn_ms(even, w, w1, w3, w2, dev, cache)
            t_nodup = _slot_ffn_ms(int(n.max()), w, w1, w3, w2, dev, cache)
            eps = float(err.item())
            rows.append({
                "workload": name, "slots": S, "extra_slots": extra, "prediction_noise": sigma,
                "prediction_error_rate": eps, "skewness_before": skew_before,
                "skewness_after": max_load / (R / S), "plan_bound": int(bound.item()), "max_slot_load": max_load,
                "even_share": even, "ffn_ms_bottleneck": t_max, "ffn_ms_even_share": t_even,
                "ffn_ms_no_duplication": t_nodup, "measured_ratio": t_max / t_even,
                "model_ratio_typical": 1.0 + eps, "speedup_vs_no_duplication": t_nodup / t_max,
            })
    return rows


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--workload", default="mixtral_skew", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--extra", type=int, nargs="+", default=[0, 2, 4, 8, 16, 24])
    ap.add_argument("--noise", type=float, nargs="+", default=[0.0, 0.1, 0.3])
    ap.add_argument("--json", action="store_true", help="one JSON object per line instead of the table")
    args = ap.parse_args()
    rows = study(args.workload, args.extra, args.noise)
    if args.json:
        for r in rows:
            print(json.dumps(r))
        return
    print(f"workload {args.workload}: skewness before the plan {rows[0]['skewness_before']:.2f}; "
          f"slot FFN without duplication {rows[0]['ffn_ms_no_duplication']:.3f} ms")
    print("| slots | noise | error rate | skewness after | bound | max load | even share | bottleneck ms | even ms |"
          " measured ratio | model 1+eps | speed-up vs no duplication |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['slots']} | {r['prediction_noise']:.2f} | {r['prediction_error_rate']:.3f} | "
              f"{r['skewness_after']:.2f} | {r['plan_bound']} | {r['max_slot_load']} | {r['even_share']} | "
              f"{r['ffn_ms_bottleneck']:.3f} | {r['ffn_ms_even_share']:.3f} | {r['measured_ratio']:.2f} | "
              f"{r['model_ratio_typical']:.2f} | {r['speedup_vs_no_duplication']:.2f} |")


if __name__ == "__main__":
    main()
