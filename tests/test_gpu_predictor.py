"""Distribution-Only predictor state and the error-rate metric on the device vs the oracle, and the
closed loop the paper describes: histogram of batch b -> predictor -> plan for batch b+1."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"


def i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


@pytest.mark.parametrize("E", [1, 8, 64, 200, 256])
def test_predictor_update_matches_oracle_over_batches(E):
    rng = np.random.default_rng(E)
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, E, 0, 1))
    state = torch.zeros(E, dtype=torch.int64, device=DEV)
    pred = torch.full((E,), -7, dtype=torch.int32, device=DEV)
    ref_state = [0] * E
    for b in range(5):
        hist = rng.integers(0, 5000, size=E)
        hist[rng.random(E) < 0.2] = 0
        ctx.predictor_update(i32(hist), state, pred)
        ref_state, ref_pred = oracle.predictor_update(ref_state, hist)
        ctx.check_status()
        assert state.cpu().tolist() == ref_state
        assert np.array_equal(pred.cpu().numpy(), ref_pred)


def test_predictor_scaling_of_huge_counts():
    E = 3
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, E, 0, 1))
    state = torch.tensor([2 ** 33, 2 ** 31, 3], dtype=torch.int64, device=DEV)
    pred = torch.zeros(E, dtype=torch.int32, device=DEV)
    ctx.predictor_update(i32([0, 0, 1]), state, pred)
    ctx.check_status()
    ref_state, ref_pred = oracle.predictor_update([2 ** 33, 2 ** 31, 3], [0, 0, 1])
    assert state.cpu().tolist() == ref_state and np.array_equal(pred.cpu().numpy(), ref_pred)
    ctx.predictor_update(i32([0, -4, 0]), state, pred)       # a negative count is reported, not added
    assert ctx.status() == binding.ERR_BAD_INDEX


@pytest.mark.parametrize("E", [4, 8, 64, 256])
def test_error_rate_matches_oracle(E):
    rng = np.random.default_rng(100 + E)
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, E, 0, 1))
    out = torch.full((1,), float("nan"), dtype=torch.float64, device=DEV)
    for _ in range(4):
        p = rng.integers(0, 10000, size=E)
        h = rng.integers(0, 10000, size=E)
        p[0] += 1
        h[-1] += 1
        ctx.error_rate(i32(p), i32(h), out)
        ref = oracle.error_rate(oracle.p_hat(p), oracle.p_hat(h))
        assert abs(out.item() - ref) <= 1e-12 * max(1.0, ref)
    ctx.error_rate(i32(h), i32(h), out)
    assert out.item() == 0.0
    if E == 4:   # the hand-worked case of the oracle's pins
        ctx.error_rate(i32([2, 2, 0, 0]), i32([1, 1, 1, 1]), out)
        assert out.item() == 1.0


def test_closed_loop_histogram_predictor_plan():
    # batch b's histogram updates the predictor whose output plans batch b+1 (paper, Section 3.1:
    # the prediction runs ahead of the layer); everything stays on the device
    T, K, E, S = 512, 2, 8, 12
    rng = np.random.default_rng(9)
    p = 1.0 / np.arange(1, E + 1) ** 1.3
    p /= p.sum()
    ctx = binding.Context(binding.Shape(T, 64, 64, E, K, S, 0, 1))
    state = torch.zeros(E, dtype=torch.int64, device=DEV)
    pred = torch.zeros(E, dtype=torch.int32, device=DEV)
    hist = torch.zeros(E, dtype=torch.int32, device=DEV)
    rep, so, se, bound = (torch.zeros(E, dtype=torch.int32, device=DEV), torch.zeros(E + 1, dtype=torch.int32, device=DEV),
                          torch.zeros(S, dtype=torch.int32, device=DEV), torch.zeros(1, dtype=torch.int32, device=DEV))
    err = torch.zeros(1, dtype=torch.float64, device=DEV)
    ref_state = [0] * E
    errors = []
    for b in range(6):
        idx = np.stack([rng.choice(E, size=K, replace=False, p=p) for _ in range(T)]).astype(np.int32)
        ctx.histogram(i32(idx), hist)
        if b > 0:
            ctx.error_rate(pred, hist, err)           # how good was the prediction made before this batch
            errors.append(err.item())
            ref_rep, _, _, ref_bound = oracle.plan(ref_pred, S)
            assert np.array_equal(rep.cpu().numpy(), ref_rep) and int(bound.item()) == ref_bound
        ctx.predictor_update(hist, state, pred)
        ctx.plan(pred, S, rep, so, se, bound)
        ref_state, ref_pred = oracle.predictor_update(ref_state, oracle.histogram(idx, E))
        ctx.check_status()
        assert np.array_equal(pred.cpu().numpy(), ref_pred)
    assert all(0.0 <= e < 0.5 for e in errors) and errors[-1] <= errors[0] + 0.05


@pytest.mark.parametrize("E,shift", [(1, 0), (8, 1), (64, 3), (256, 6), (200, 16)])
def test_predictor_update_ema_matches_oracle_over_batches(E, shift):
    rng = np.random.default_rng(7 * E + shift)
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, E, 0, 1))
    state = torch.zeros(E, dtype=torch.int64, device=DEV)
    pred = torch.full((E,), -7, dtype=torch.int32, device=DEV)
    ref_state = [0] * E
    for b in range(8):
        hist = rng.integers(0, 2 ** 31 - 1 if b == 3 else 60000, size=E)     # one batch of huge counts: the scaling path
        hist[rng.random(E) < 0.2] = 0
        ctx.predictor_update_ema(i32(hist), state, shift, pred)
        ref_state, ref_pred = oracle.predictor_update_ema(ref_state, hist, shift)
        ctx.check_status()
        assert state.cpu().tolist() == ref_state
        assert np.array_equal(pred.cpu().numpy(), ref_pred)
    with pytest.raises(binding.MoegpsError):
        ctx.predictor_update_ema(i32(hist), state, 17, pred)


def test_layer_replans_every_n_batches_from_the_predictor():
    """The loop of Section 3.1 with a chosen prediction / placement frequency: every batch updates the
    predictor state from its own histogram; every n-th batch the plan is renewed from the prediction."""
    from paper_2506_07366_b200 import workloads as wl
    from paper_2506_07366_b200.layer import MoeLayer
    w = wl.WORKLOADS["tiny"].scaled(S=12)
    wr, bias = wl.router(w, DEV)
    w1, w3, w2 = wl.expert_weights(w, DEV)
    shape = binding.Shape(w.T, w.D, w.F, w.E, w.K, w.S, w.gate_mode, 128)
    for every, shift in ((1, None), (3, None), (2, 2)):
        layer = MoeLayer(shape, wr, bias, w1, w3, w2)
        layer.start_prediction(replan_every=every, ema_shift=shift)
        ref_state, ref_pred = [0] * w.E, np.zeros(w.E, dtype=np.int32)
        ref_rep = oracle.plan(ref_pred, w.S)[0]
        for b in range(7):
            x = wl.activations(w.scaled(number=w.number + 11 * b), DEV)
            assert np.array_equal(layer.replicas.cpu().numpy(), ref_rep), (every, shift, b)   # the plan batch b runs under
            layer.forward_predicted(x)
            layer.ctx.check_status()
            hist = layer.hist.cpu().numpy()
            if shift is None:
                ref_state, ref_pred = oracle.predictor_update(ref_state, hist)
            else:
                ref_state, ref_pred = oracle.predictor_update_ema(ref_state, hist, shift)
            if (b + 1) % every == 0:
                ref_rep = oracle.plan(ref_pred, w.S)[0]
        assert np.array_equal(layer.replicas.cpu().numpy(), ref_rep)
