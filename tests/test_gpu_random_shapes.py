"""Seeded sweep of small, awkward layer shapes through the whole path against the oracle: dimensions
that are not multiples of any tile, single tokens, single experts, K = E, many empty slots, a copy
cap, every row alignment.  Each case is compared element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding, workloads as wl
from paper_2506_07366_b200.layer import MoeLayer
from tests import harness as hz

pytestmark = pytest.mark.gpu
DEV = "cuda"


def random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        E = int(rng.choice([1, 2, 3, 5, 8, 17, 33, 64]))
        K = int(rng.integers(1, min(E, 8) + 1))
        cases.append(dict(
            T=int(rng.choice([1, 2, 7, 31, 128, 129, 300, 555])), D=int(8 * rng.integers(1, 66)),
            F=int(8 * rng.integers(1, 50)), E=E, K=K, S=int(E + rng.integers(0, 21)),
            gate_mode=int(rng.integers(0, 2)), A=int(rng.choice([1, 8, 128])), c_max=int(rng.choice([0, 0, 2])),
            zipf=float(rng.choice([0.0, 1.0, 2.0])), seed=1000 + i))
    return cases


@pytest.mark.parametrize("c", random_cases(16, 20250607), ids=lambda c: "T{T}-D{D}-F{F}-E{E}-K{K}-S{S}-A{A}-c{c_max}".format(**c))
def test_random_layer_shape(c):
    w = wl.Workload("random", c["seed"], T=c["T"], D=c["D"], F=c["F"], E=c["E"], K=c["K"], S=c["S"],
                    gate_mode=c["gate_mode"], zipf_s=c["zipf"], sigma_x=1.0, prediction="noisy")
    wr, bias = wl.router(w, "cpu")
    x, _ = hz.screened_activations(w, wr, bias)
    w1, w3, w2 = wl.expert_weights(w, "cpu")
    w1, w3, w2 = (w1.float() * 8).bfloat16(), (w3.float() * 8).bfloat16(), (w2.float() * 8).bfloat16()
    true_hist = oracle.histogram(oracle.route(hz.bits(x), hz.bits(wr), bias.numpy(), w.K, w.gate_mode)[0], w.E)
    pred = wl.noisy_prediction(w, torch.from_numpy(true_hist)).numpy()
    ref = oracle.moe_layer(hz.bits(x), hz.bits(wr), bias.numpy(), hz.bits(w1), hz.bits(w3), hz.bits(w2), pred,
                           K=w.K, S=w.S, gate_mode=w.gate_mode, row_align=c["A"], c_max=c["c_max"])
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, c["A"], c["c_max"])
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer.out.fill_(float("nan"))
    layer.xp.fill_(float("nan"))                       # padding rows stay NaN and must not leak
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
