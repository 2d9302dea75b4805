"""Whole-layer parity: MoeLayer (route -> histogram -> plan -> dispatch -> expert_ffn -> combine
through the C ABI) against the oracle.

Small and scaled-down workloads are compared element by element.  The full-size workloads are run
in the launch configuration the benchmark times; their integer steps are compared exactly over the
whole batch, and their float outputs either over the whole batch (where the oracle needs seconds)
or on the first and last occupied row of every row tile of every slot.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding, workloads as wl
from paper_2506_07366_b200.layer import MoeLayer, ROW_ALIGN
from tests import harness as hz

pytestmark = pytest.mark.gpu
DEV = "cuda"

SMALL = [
    (wl.WORKLOADS["tiny"], 128),
    (wl.WORKLOADS["tiny"], 1),
    (wl.WORKLOADS["mixtral"].scaled(T=384, D=512, F=1792), 128),
    (wl.WORKLOADS["mixtral_skew"].scaled(T=1024, D=256, F=896), 128),
    (wl.WORKLOADS["many_expert"].scaled(T=512, D=256, F=352), 128),
    (wl.WORKLOADS["fine_grained"].scaled(T=256, D=448, F=128), 128),
    (wl.WORKLOADS["fine_grained"].scaled(T=256, D=448, F=128), 16),
]


def build_inputs(w, device):
    wr, bias = wl.router(w, "cpu")
    x, _ = hz.screened_activations(w, wr, bias)
    w1, w3, w2 = wl.expert_weights(w, "cpu")
    return x, wr, bias, w1, w3, w2


@pytest.mark.parametrize("w,A", SMALL, ids=lambda v: v if isinstance(v, int) else f"{v.name}-T{v.T}")
def test_layer_small(w, A):
    x, wr, bias, w1, w3, w2 = build_inputs(w, DEV)
    ref_idx, _, _ = oracle.route(hz.bits(x), hz.bits(wr), bias.numpy(), w.K, w.gate_mode)
    pred = hz.predicted_histogram(w, oracle.histogram(ref_idx, w.E), wr, bias)
    ref = oracle.moe_layer(hz.bits(x), hz.bits(wr), bias.numpy(), hz.bits(w1), hz.bits(w3), hz.bits(w2), pred,
                           K=w.K, S=w.S, gate_mode=w.gate_mode, row_align=A)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, A)
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer.out.fill_(float("nan"))
    layer.plan(torch.from_numpy(pred))
    out = layer.forward(x.to(DEV))
    layer.ctx.check_status()
    for name in ("replicas", "slot_off", "slot_expert", "topk_idx", "hist", "slot_row_off", "row_pair", "pair_row"):
        assert np.array_equal(getattr(layer, name).cpu().numpy(), ref[name]), name
    assert int(layer.bound.item()) == ref["bound"]
    hz.assert_close_rel_max(layer.topk_w.cpu().numpy(), ref["topk_w"], "topk_w")
    occ = ref["row_pair"] >= 0
    assert np.array_equal(hz.bits(layer.xp)[occ], ref["xp"][occ])
    hz.assert_close_rel_max(layer.yp.float().cpu().numpy()[occ], ref["yp"][occ], "yp")
    hz.assert_close_rel_max(out.float().cpu().numpy(), ref["out"], "out")
    # placement never changes results: same layer without duplication (S = E), compact rows
    shape2 = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.E, w.gate_mode, 1)
    layer2 = MoeLayer(shape2, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer2.plan(torch.zeros(w.E, dtype=torch.int32))
    out2 = layer2.forward(x.to(DEV))
    layer2.ctx.check_status()
    assert torch.equal(out2, out)      # same rows, same arithmetic order => bitwise equal


def test_layer_host_buffers():
    w = wl.WORKLOADS["tiny"]
    x, wr, bias, w1, w3, w2 = build_inputs(w, DEV)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, 128)
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer.plan(torch.ones(w.E, dtype=torch.int32))
    xh = x.pin_memory()
    oh = torch.empty(w.T, w.D, dtype=torch.bfloat16).pin_memory()
    layer.forward_host(xh, oh)
    torch.cuda.synchronize()
    assert torch.equal(oh, layer.forward(x.to(DEV)).cpu())


def test_host_pipeline_overlapped_copies_give_the_same_results():
    from paper_2506_07366_b200.layer import HostPipeline
    w = wl.WORKLOADS["tiny"]
    _, wr, bias, w1, w3, w2 = build_inputs(w, DEV)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, 128)
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer.plan(torch.ones(w.E, dtype=torch.int32))
    batches = [wl.activations(w.scaled(number=w.number + 7 * i), "cpu").pin_memory() for i in range(5)]
    outs = [torch.zeros(w.T, w.D, dtype=torch.bfloat16).pin_memory() for _ in batches]
    pipe = HostPipeline(layer, depth=2)
    for xb, ob in zip(batches, outs):
        pipe.submit(xb, ob)
    pipe.drain()
    torch.cuda.synchronize()
    layer.ctx.check_status()
    for xb, ob in zip(batches, outs):
        assert torch.equal(ob, layer.forward(xb.to(DEV)).cpu())


def test_captured_graph_replays_the_step_on_new_inputs():
    w = wl.WORKLOADS["tiny"]
    _, wr, bias, w1, w3, w2 = build_inputs(w, DEV)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S + 3, w.gate_mode, 128)
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    x = wl.activations(w, DEV)
    pred = torch.ones(w.E, dtype=torch.int32, device=DEV)
    graph = layer.capture(x, pred)
    for i in range(3):
        x.copy_(wl.activations(w.scaled(number=w.number + 3 + i), DEV))      # new batch, same buffers
        pred.copy_(torch.randint(0, 100, (w.E,), dtype=torch.int32, device=DEV))
        graph.replay()
        torch.cuda.synchronize()
        got, got_rep = layer.out.clone(), layer.replicas.clone()
        layer.plan(pred)
        want = layer.forward(x).clone()
        layer.ctx.check_status()
        assert torch.equal(got, want) and torch.equal(got_rep, layer.replicas)


class ExpertsOnDemand:
    """w[e] -> host bf16 bits of one expert's matrix, fetched from the device when asked for."""

    def __init__(self, t):
        self.t = t

    def __getitem__(self, e):
        return hz.bits(self.t[int(e)])


# name -> how the float outputs are compared at full size:
#   "all"   every occupied row of yp and every token of out (the oracle needs seconds for these)
#   "tiles" the first and the last occupied row of EVERY 128-row stretch of every slot for yp - so a
#           defect confined to one row tile, one slot or one round of the persistent tile loop shows -
#           and out on the tokens that own a seeded subset of those rows
FULL = [("mixtral", "all"), ("mixtral_skew", "tiles"), ("many_expert", "all"), ("fine_grained", "tiles")]
MAX_OUT_TOKENS = 96


@pytest.mark.parametrize("name,coverage", FULL, ids=[n for n, _ in FULL])
def test_layer_full_size(name, coverage):
    w = wl.WORKLOADS[name]
    torch.cuda.empty_cache()
    wr, bias = wl.router(w, DEV)
    x0 = wl.activations(w, DEV)
    x, redrawn = hz.screened_activations(w, wr.cpu(), bias.cpu(), x0.cpu())
    assert redrawn <= 0.05 * w.T
    w1, w3, w2 = wl.expert_weights(w, DEV)
    xb, wrb, bb = hz.bits(x), hz.bits(wr), bias.cpu().numpy()
    ref_idx, ref_w, ref_logits = oracle.route(xb, wrb, bb, w.K, w.gate_mode)
    ref_hist = oracle.histogram(ref_idx, w.E)
    pred = hz.predicted_histogram(w, ref_hist, wr.cpu(), bias.cpu())
    A = ROW_ALIGN                                   # the launch configuration the benchmark times
    rep, so, se, bound = oracle.plan(pred, w.S)
    sro, rp, pr, _ = oracle.dispatch(None, ref_idx, ref_hist, rep, so, w.S, A)

    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, A)
    layer = MoeLayer(shape, wr, bias, w1, w3, w2)
    layer.plan(torch.from_numpy(pred))
    xd = x.to(DEV)
    out = layer.forward(xd)
    layer.ctx.check_status()
    logits = torch.empty(w.T, w.E, dtype=torch.float32, device=DEV)
    layer.ctx.route_logits(xd, wr, bias, logits)
    assert np.abs(logits.cpu().numpy().astype(np.float64) - ref_logits).max() < hz.TAU / 4

    # integer steps: exact over the whole batch
    assert np.array_equal(layer.topk_idx.cpu().numpy(), ref_idx)
    assert np.array_equal(layer.hist.cpu().numpy(), ref_hist)
    assert np.array_equal(layer.replicas.cpu().numpy(), rep)
    assert np.array_equal(layer.slot_off.cpu().numpy(), so)
    assert np.array_equal(layer.slot_expert.cpu().numpy(), se)
    assert int(layer.bound.item()) == bound
    assert np.array_equal(layer.slot_row_off.cpu().numpy(), sro)
    assert np.array_equal(layer.row_pair.cpu().numpy(), rp)
    assert np.array_equal(layer.pair_row.cpu().numpy(), pr)
    hz.assert_close_rel_max(layer.topk_w.cpu().numpy(), ref_w, "topk_w")
    # properties that hold at any size, checked on the device results
    assert int(layer.hist.sum()) == w.T * w.K
    rows = layer.pair_row.reshape(-1).long()
    assert torch.equal(layer.row_pair[rows].long(), torch.arange(w.R, device=DEV))
    assert torch.equal(layer.xp[rows], xd.repeat_interleave(w.K, dim=0))       # rows are bit copies
    loads = np.diff(sro)
    assert loads.max() <= -(-int(np.ceil(max(1.0, (ref_hist / np.maximum(pred, 1)).max()) * bound)) // A) * A
    assert torch.isfinite(out.float()).all()

    # float outputs
    experts = [ExpertsOnDemand(t) for t in (w1, w3, w2)]
    if coverage == "all":
        yp_rows = np.nonzero(rp >= 0)[0]
        tokens = np.arange(w.T)
    else:
        picked = []
        for s in range(w.S):
            n_occ = int(np.count_nonzero(rp[sro[s]:sro[s + 1]] >= 0))       # occupied rows lead the slot
            for lo in range(0, n_occ, 128):
                picked += [sro[s] + lo, sro[s] + min(lo + 128, n_occ) - 1]
        yp_rows = np.unique(np.array(picked, dtype=np.int64))
        assert (rp[yp_rows] >= 0).all()
        rng = np.random.default_rng(w.seed)
        owners = np.unique(rp[yp_rows] // w.K)
        tokens = np.sort(rng.choice(owners, size=min(MAX_OUT_TOKENS, owners.size), replace=False))
    need = np.unique(np.concatenate([yp_rows, pr[tokens].reshape(-1)]))
    xp_bits = np.zeros((shape.Rcap, w.D), dtype=np.uint16)
    xp_bits[need] = xb[rp[need] // w.K]
    yp_ref = oracle.expert_ffn(xp_bits, sro, se, *experts, rows=need)
    out_ref = oracle.combine(yp_ref, pr, ref_w, tokens=tokens)
    yp_got = layer.yp[torch.from_numpy(need).to(DEV)].float().cpu().numpy()
    hz.assert_close_rel_max(yp_got, yp_ref[need], f"yp ({need.size} rows)")
    out_got = out[torch.from_numpy(tokens).to(DEV)].float().cpu().numpy()
    hz.assert_close_rel_max(out_got, out_ref[tokens], f"out ({tokens.size} tokens)")


def test_plan_study_runs_on_a_small_workload():
    """The plan-quality script end to end on the tiny workload: more replica slots never raise the
    bottleneck load under an exact prediction, and the reported loads respect the planner's bound."""
    from paper_2506_07366_b200 import plan_study
    rows = plan_study.study("tiny", extras=[0, 2, 4], noises=[0.0])
    assert [r["slots"] for r in rows] == [8, 10, 12]
    loads = [r["max_slot_load"] for r in rows]
    assert loads == sorted(loads, reverse=True)
    for r in rows:
        assert r["max_slot_load"] == r["plan_bound"]          # exact prediction: the split realises the plan
        assert r["prediction_error_rate"] == 0.0
        assert r["ffn_ms_bottleneck"] > 0 and r["ffn_ms_even_share"] > 0
        assert r["ffn_ms_whole_layer_one_device"] > 0
    # a copy cap of 2 (Algorithm 1's C_max) leaves slots empty once every expert worth copying has two
    capped = plan_study.study("tiny", extras=[12], noises=[0.0], c_maxes=[0, 2], in_situ=False)
    assert capped[0]["slots_used"] == 20 and capped[1]["slots_used"] == 16
    assert capped[1]["max_slot_load"] >= capped[0]["max_slot_load"]
