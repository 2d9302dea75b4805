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
                                             [--c-max 0 2 3] [--out FILE]

`--c-max` sweeps Algorithm 1's cap on the copies of one expert; the `layer ms` column is expert_ffn of
the whole dispatched batch on this one device, next to the isolated-slot times.

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


def _slot_loads(slot_row_off, row_pair, rcap):
    """Rows that carry a pair, per slot (slot extents are padded to the row alignment)."""
    occupied = (row_pair >= 0).to(torch.int64).cumsum(0)
    ends = slot_row_off[1:].long().clamp(max=rcap) - 1
    starts = slot_row_off[:-1].long() - 1
    at = lambda i: torch.where(i >= 0, occupied[i.clamp(min=0)], torch.zeros_like(i))  # noqa: E731
    return (at(ends) - at(starts)).cpu()


def study(name: str, extras, noises, c_maxes=(0,), in_situ=True, device=0):
    """One row per (extra slots, copy cap, prediction noise).  `in_situ` also times the whole layer's
    expert_ffn on the dispatched batch (all slots on this one device, all experts' weights)."""
    torch.cuda.set_device(device)
    dev = torch.device("cuda", device)
    w = wl.WORKLOADS[name]
    wr, bias = wl.router(w, dev)
    x = wl.activations(w, dev)
    if in_situ:
        w1, w3, w2 = wl.expert_weights(w, dev)
    else:
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
    stream = torch.cuda.current_stream()
    for extra in extras:
        S = w.E + extra
        for c_max in c_maxes:
            shape = Shape(w.T, w.D, w.F, w.E, w.K, S, w.gate_mode, 128, c_max)
            ctx = Context(shape)
            replicas, slot_off = torch.empty(w.E, **i32), torch.empty(w.E + 1, **i32)
            slot_expert, bound = torch.empty(S, **i32), torch.empty(1, **i32)
            slot_row_off, row_pair = torch.empty(S + 1, **i32), torch.empty(shape.Rcap, **i32)
            pair_row = torch.empty(w.T, w.K, **i32)
            xp = torch.empty(shape.Rcap, w.D, dtype=torch.bfloat16, device=dev)
            ws = torch.empty(max(16, workspace_bytes(shape)), dtype=torch.uint8, device=dev)
            err = torch.zeros(1, dtype=torch.float64, device=dev)
            if in_situ:
                h_ws = torch.empty(shape.Rcap, w.F, dtype=torch.bfloat16, device=dev)
                yp = torch.empty(shape.Rcap, w.D, dtype=torch.bfloat16, device=dev)
            for sigma in noises:
                g = torch.Generator(device="cpu")
                g.manual_seed(w.seed + 6 + int(1000 * sigma))
                z = torch.randn(w.E, generator=g, dtype=torch.float64)
                pred = torch.clamp(torch.round(n * (1.0 + sigma * z)), min=0).to(torch.int32).to(dev)
                ctx.plan(pred, S, replicas, slot_off, slot_expert, bound)
                ctx.dispatch(x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp, ws)
                ctx.error_rate(pred, hist, err)
                ctx.check_status()
                loads = _slot_loads(slot_row_off, row_pair, shape.Rcap)
                used_slots = int((slot_expert >= 0).sum())
                max_load, even = int(loads.max()), -(-R // S)
                t_max = _slot_ffn_ms(max_load, w, w1, w3, w2, dev, cache)
                t_even = _slot_ffn_ms(even, w, w1, w3, w2, dev, cache)
                t_nodup = _slot_ffn_ms(int(n.max()), w, w1, w3, w2, dev, cache)
                t_layer = None
                if in_situ:
                    times = []
                    for i in range(5):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record(stream)
                        ctx.expert_ffn(xp, slot_row_off, slot_expert, w1, w3, w2, h_ws, yp)
                        e1.record(stream)
                        e1.synchronize()
                        if i >= 2:
                            times.append(e0.elapsed_time(e1))
                    ctx.check_status()
                    t_layer = statistics.median(times)
                eps = float(err.item())
                skew_after = max_load / (R / S)
                rows.append({
                    "workload": name, "slots": S, "extra_slots": extra, "c_max": c_max, "slots_used": used_slots,
                    "prediction_noise": sigma, "prediction_error_rate": eps, "skewness_before": skew_before,
                    "skewness_after": skew_after, "plan_bound": int(bound.item()), "max_slot_load": max_load,
                    "even_share": even, "ffn_ms_bottleneck": t_max, "ffn_ms_even_share": t_even,
                    "ffn_ms_no_duplication": t_nodup, "measured_ratio": t_max / t_even,
                    # the paper's two models of that ratio: the bottleneck device is slower than the even
                    # share by the skewness that is left (Section 2), and after prediction-driven
                    # duplication by 1 + error rate in the typical case (Section 3.3)
                    "model_ratio_skewness": skew_after, "model_ratio_typical": 1.0 + eps,
                    "speedup_vs_no_duplication": t_nodup / t_max, "ffn_ms_whole_layer_one_device": t_layer,
                })
    return rows


def render(rows, argv) -> str:
    r0 = rows[0]
    out = [f"# Plan-quality study, workload `{r0['workload']}`, one B200", "",
           "    python -m paper_2506_07366_b200.plan_study " + " ".join(argv), "",
           f"Skewness before the plan {r0['skewness_before']:.2f}; the most loaded expert alone (no duplication) needs "
           f"{r0['ffn_ms_no_duplication']:.3f} ms of expert_ffn.  `bottleneck ms` / `even ms`: expert_ffn of ONE slot "
           "holding the largest slot load / the even share R/S (a slot stands for a device of the paper's "
           "expert-parallel deployment); `ratio` = their quotient, next to the paper's models of it: the skewness left "
           "after duplication (Section 2) and 1 + error rate (typical case, Section 3.3).  `layer ms` = expert_ffn of "
           "the whole dispatched batch on this one device (placement changes where rows sit, not how much work there is).",
           "",
           "| slots | c_max | slots used | noise | error rate | skewness after | bound | max load | even share | "
           "bottleneck ms | even ms | ratio | model: skewness | model: 1+eps | speed-up vs no duplication | layer ms |",
           "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        layer = "-" if r["ffn_ms_whole_layer_one_device"] is None else f"{r['ffn_ms_whole_layer_one_device']:.3f}"
        out.append(f"| {r['slots']} | {r['c_max']} | {r['slots_used']} | {r['prediction_noise']:.2f} | "
                   f"{r['prediction_error_rate']:.3f} | {r['skewness_after']:.2f} | {r['plan_bound']} | "
                   f"{r['max_slot_load']} | {r['even_share']} | {r['ffn_ms_bottleneck']:.3f} | "
                   f"{r['ffn_ms_even_share']:.3f} | {r['measured_ratio']:.2f} | {r['model_ratio_skewness']:.2f} | "
                   f"{r['model_ratio_typical']:.2f} | {r['speedup_vs_no_duplication']:.2f} | {layer} |")
    return "\n".join(out) + "\n"


def main():
    import sys
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--workload", default="mixtral_skew", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--extra", type=int, nargs="+", default=[0, 2, 4, 8, 16, 24])
    ap.add_argument("--noise", type=float, nargs="+", default=[0.0, 0.1, 0.3])
    ap.add_argument("--c-max", type=int, nargs="+", default=[0], help="copy caps to sweep (Algorithm 1's C_max; 0 = none)")
    ap.add_argument("--no-in-situ", action="store_true", help="skip the whole-layer expert_ffn timing")
    ap.add_argument("--json", action="store_true", help="one JSON object per line instead of the table")
    ap.add_argument("--out", help="also write the table (markdown, with this command line) to this file")
    args = ap.parse_args()
    rows = study(args.workload, args.extra, args.noise, args.c_max, not args.no_in_situ)
    if args.json:
        for r in rows:
            print(json.dumps(r))
        return
    text = render(rows, [a for a in sys.argv[1:] if a != "--out" and a != args.out])
    print(text, end="")
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
