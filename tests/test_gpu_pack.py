"""moegps_pack (Algorithm 1 on G devices with limited memory) against the oracle: the sequence of
moves is deterministic (fixed tie-breaks), so placement, shares, loads and the number of moves must
all match exactly."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"


def i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def run_pack(n, home, cap, c_max):
    E, G = len(n), len(cap)
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, E, 0, 1, c_max))
    placed = torch.full((E, G), -7, dtype=torch.int32, device=DEV)
    share = torch.full((E, G), -7, dtype=torch.int32, device=DEV)
    load = torch.full((G,), -7, dtype=torch.int32, device=DEV)
    iters = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    ctx.pack(i32(n), i32(home), i32(cap), G, placed, share, load, iters)
    return ctx, placed.cpu().numpy(), share.cpu().numpy(), load.cpu().numpy(), int(iters.item())


def check(n, home, cap, c_max):
    ctx, placed, share, load, iters = run_pack(n, home, cap, c_max)
    ctx.check_status()
    p_ref, s_ref, l_ref, it_ref = oracle.pack(n, home, cap, c_max)
    assert np.array_equal(placed, p_ref)
    assert np.array_equal(share, s_ref)
    assert np.array_equal(load, l_ref)
    assert iters == it_ref
    return iters


HAND = [
    ([9, 1, 1, 1], [0, 1, 2, 3], [4, 4, 4, 4], 0),        # the paper's four-GPU example
    ([5, 0], [0, 1], [2, 2], 0), ([4, 4, 0, 0], [0, 1, 2, 3], [2, 2, 2, 2], 0), ([3, 3, 1], [0, 0, 0], [3, 3], 0),
    ([7, 2], [0, 0], [2], 0), ([3, 4], [0, 1], [2, 2], 0), ([1000, 10, 10, 10], [0, 1, 2, 3], [4] * 4, 1),
    ([1000, 10, 10, 10], [0, 1, 2, 3], [4] * 4, 2), ([1000, 10, 10, 10], [0, 1, 2, 3], [1] * 4, 0),
    ([100], [0], [1, 1, 1], 0), ([0, 0, 0], [2, 1, 0], [1, 1, 1], 0), ([2 ** 31 - 6, 5], [0, 1], [2, 2], 0),
]


@pytest.mark.parametrize("n,home,cap,c_max", HAND)
def test_pack_hand_cases(n, home, cap, c_max):
    check(np.array(n, dtype=np.int64), home, cap, c_max)


@pytest.mark.parametrize("E,G,skew,slack,c_max,seed", [
    (8, 4, 1.5, 2, 0, 0), (8, 8, 0.8, 1, 0, 1), (64, 8, 1.2, 2, 0, 2), (64, 16, 1.2, 1, 3, 3),
    (256, 8, 1.0, 4, 0, 4), (256, 32, 1.0, 1, 0, 5), (256, 64, 1.0, 2, 4, 6), (200, 37, 2.0, 0, 0, 7),
    (33, 33, 0.0, 1, 2, 8), (1, 5, 0.0, 1, 0, 9), (256, 64, 1.0, 0, 0, 10),
])
def test_pack_random(E, G, skew, slack, c_max, seed):
    rng = np.random.default_rng(seed)
    p = 1.0 / np.arange(1, E + 1) ** skew
    n = rng.multinomial(32768, p / p.sum())
    rng.shuffle(n)
    home = rng.integers(0, G, size=E)
    cap = np.bincount(home, minlength=G) + slack + rng.integers(0, 2, size=G) * (slack > 0)
    iters = check(n, home, cap, c_max)
    if slack > 0 and c_max == 0 and E >= 8:
        assert iters > 0


def test_pack_reports_bad_inputs_without_faulting():
    ctx, placed, share, load, iters = run_pack(np.array([5, 5, 5]), [0, 7, 1], [2, 2], 0)      # home out of range
    assert ctx.status() == binding.ERR_BAD_INDEX and iters == 0
    ctx, placed, share, load, iters = run_pack(np.array([5, 5, 5]), [0, 0, 0], [2, 3], 0)      # device 0 over-full
    assert ctx.status() == binding.ERR_BAD_INDEX and iters == 0
    ctx, placed, share, load, iters = run_pack(np.array([2 ** 31 - 1, 5]), [0, 1], [2, 2], 0)  # loads would not fit int32
    assert ctx.status() == binding.ERR_BAD_INDEX and iters == 0
    ctx = binding.Context(binding.Shape(8, 64, 64, 4, 1, 4, 0, 1))
    with pytest.raises(binding.MoegpsError) as ei:                                                # too many devices
        ctx.pack(i32([1] * 4), i32([0] * 4), i32([4] * 65), 65, torch.zeros(4, 65, dtype=torch.int32, device=DEV),
                 torch.zeros(4, 65, dtype=torch.int32, device=DEV), torch.zeros(65, dtype=torch.int32, device=DEV),
                 torch.zeros(1, dtype=torch.int32, device=DEV))
    assert ei.value.code == binding.ERR_UNSUPPORTED_SHAPE


def pack_and_slots_on_device(ctx, n, home, cap, S):
    E, G = len(n), len(cap)
    i32z = lambda *shape: torch.full(shape, -7, dtype=torch.int32, device=DEV)  # noqa: E731
    placed, share, load, iters = i32z(E, G), i32z(E, G), i32z(G), i32z(1)
    ctx.pack(i32(n), i32(home), i32(cap), G, placed, share, load, iters)
    rep, so, se, ss, sd = i32z(E), i32z(E + 1), i32z(S), i32z(S), i32z(S)
    ctx.pack_slots(placed, share, G, rep, so, se, ss, sd)
    return placed, share, load, rep, so, se, ss, sd


@pytest.mark.parametrize("E,G,K,T,A,D,seed", [
    (6, 3, 2, 300, 4, 64, 0), (8, 4, 2, 1000, 128, 128, 1), (64, 8, 6, 777, 16, 64, 2), (256, 16, 8, 515, 1, 128, 3),
    (16, 5, 6, 45000, 16, 16, 4),          # more than 1024 segments: the path that scans the counts on the device
])
def test_pack_slots_and_dispatch_shares_match_the_oracle(E, G, K, T, A, D, seed):
    rng = np.random.default_rng(seed)
    logp = -1.2 * np.log(np.arange(1, E + 1))
    idx = np.argsort(-(logp[None, :] + rng.gumbel(size=(T, E))), axis=1)[:, :K].astype(np.int32)
    hist = oracle.histogram(idx, E)
    pred = np.maximum(0, np.round(hist * (1 + 0.2 * rng.normal(size=E)))).astype(np.int64)
    pred[rng.integers(0, E)] = 0                                     # one expert the prediction missed entirely
    home = rng.integers(0, G, size=E)
    cap = np.bincount(home, minlength=G) + 3
    p_ref, s_ref, l_ref, _ = oracle.pack(pred, home, cap)
    S = int(p_ref.sum()) + 5
    rep_ref, so_ref, se_ref, ss_ref, sd_ref = oracle.pack_slots(p_ref, s_ref, S)
    shape = binding.Shape(T, D, 64, E, K, S, 0, A)
    ctx = binding.Context(shape)
    placed, share, load, rep, so, se, ss, sd = pack_and_slots_on_device(ctx, pred, home, cap, S)
    ctx.check_status()
    for got, want in ((placed, p_ref), (share, s_ref), (load, l_ref), (rep, rep_ref), (so, so_ref), (se, se_ref),
                      (ss, ss_ref), (sd, sd_ref)):
        assert np.array_equal(got.cpu().numpy(), want)
    x = rng.integers(0, 1 << 15, size=(T, D), dtype=np.uint16)
    sro_ref, rp_ref, pr_ref, xp_ref = oracle.dispatch(x, idx, hist, rep_ref, so_ref, S, A, slot_share=ss_ref)
    sro = torch.full((S + 1,), -7, dtype=torch.int32, device=DEV)
    rp = torch.full((shape.Rcap,), -7, dtype=torch.int32, device=DEV)
    pr = torch.full((T, K), -7, dtype=torch.int32, device=DEV)
    xp = torch.full((shape.Rcap, D), 0x5A5A, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    ws = torch.full((binding.workspace_bytes(shape),), 0xFF, dtype=torch.uint8, device=DEV)
    xd = torch.from_numpy(x.view(np.int16).copy()).view(torch.bfloat16).to(DEV)
    ctx.dispatch_shares(xd, i32(idx), i32(hist), rep, so, ss, sro, rp, pr, xp, ws)
    ctx.check_status()
    assert np.array_equal(sro.cpu().numpy(), sro_ref)
    assert np.array_equal(rp.cpu().numpy(), rp_ref)
    assert np.array_equal(pr.cpu().numpy(), pr_ref)
    occ = rp_ref >= 0
    got_xp = xp.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got_xp[occ], xp_ref[occ]) and (got_xp[~occ] == 0x5A5A).all()
    # what the placement is for: loads per device, realised on the actual routing
    loads = np.array([np.count_nonzero(rp_ref[sro_ref[s]:sro_ref[s + 1]] >= 0) for s in range(S)])
    per_device = np.array([loads[sd_ref == g].sum() for g in range(G)])
    assert per_device.sum() == T * K


def test_pack_slots_reports_too_few_slots():
    E, G = 4, 2
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, 5, 0, 1))                      # 5 slots
    placed = i32(np.ones((E, G)))                                                        # 8 copies
    share = i32(np.ones((E, G)))
    outs = [torch.zeros(n, dtype=torch.int32, device=DEV) for n in (E, E + 1, 5, 5, 5)]
    ctx.pack_slots(placed, share, G, *outs)
    assert ctx.status() == binding.ERR_BAD_INDEX


def test_layer_under_a_packed_placement_equals_the_oracle():
    """plan by moegps_pack on 4 devices -> slot tables -> route -> dispatch by shares -> expert_ffn ->
    combine: integers exact, floats within tolerance; and the output does not depend on the placement."""
    from paper_2506_07366_b200 import workloads as wl
    from paper_2506_07366_b200.layer import MoeLayer
    from tests import harness as hz
    w = wl.WORKLOADS["tiny"]
    G = 4
    wr, bias = wl.router(w, "cpu")
    x, _ = hz.screened_activations(w, wr, bias)
    w1, w3, w2 = wl.expert_weights(w, "cpu")
    bits = hz.bits
    ref_idx, ref_w, _ = oracle.route(bits(x), bits(wr), bias.numpy(), w.K, w.gate_mode)
    hist = oracle.histogram(ref_idx, w.E)
    pred = hz.predicted_histogram(w, hist, wr, bias)
    home = np.arange(w.E) % G
    cap = np.full(G, w.E // G + 2)
    p_ref, s_ref, l_ref, _ = oracle.pack(pred, home, cap)
    S = int(cap.sum())
    rep, so, se, ss, sd = oracle.pack_slots(p_ref, s_ref, S)
    A = 16
    sro, rp, pr, xp = oracle.dispatch(bits(x), ref_idx, hist, rep, so, S, A, slot_share=ss)
    yp = oracle.expert_ffn(xp, sro, se, bits(w1), bits(w3), bits(w2))
    out_ref = oracle.combine(yp, pr, ref_w)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, S, w.gate_mode, A)
    layer = MoeLayer(shape, wr.to(DEV), bias.to(DEV), w1.to(DEV), w3.to(DEV), w2.to(DEV))
    ctx = layer.ctx
    placed, share, load, d_rep, d_so, d_se, d_ss, d_sd = pack_and_slots_on_device(ctx, pred, home, cap, S)
    xd = x.to(DEV)
    ctx.route_histogram(xd, layer.w_router, layer.bias, layer.topk_idx, layer.topk_w, layer.hist)
    ctx.dispatch_shares(xd, layer.topk_idx, layer.hist, d_rep, d_so, d_ss, layer.slot_row_off, layer.row_pair,
                        layer.pair_row, layer.xp, layer.workspace)
    ctx.expert_ffn(layer.xp, layer.slot_row_off, d_se, layer.w_gate, layer.w_up, layer.w_down, layer.h_ws, layer.yp)
    ctx.combine(layer.yp, layer.pair_row, layer.topk_w, layer.out)
    ctx.check_status()
    assert np.array_equal(layer.topk_idx.cpu().numpy(), ref_idx)
    assert np.array_equal(layer.slot_row_off.cpu().numpy(), sro)
    assert np.array_equal(layer.pair_row.cpu().numpy(), pr)
    hz.assert_close_rel_max(layer.out.float().cpu().numpy(), out_ref, "out")
    # same batch under the slot planner's placement: same rows, same arithmetic per row
    layer2 = MoeLayer(binding.Shape(w.T, w.D, w.F, w.E, w.K, w.E, w.gate_mode, 1), wr.to(DEV), bias.to(DEV),
                      w1.to(DEV), w3.to(DEV), w2.to(DEV))
    layer2.plan(torch.zeros(w.E, dtype=torch.int32))
    assert torch.equal(layer2.forward(xd), layer.out)
