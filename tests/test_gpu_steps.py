"""Per-step parity of the CUDA kernels (through the C ABI) with the CPU oracle.

Each step is fed the ORACLE's inputs for that step, so a defect in one kernel cannot hide behind, or
be blamed on, another.  Integers must match exactly; floats within 2e-2 * max|ref| (tighter where
the arithmetic allows it).  Outputs are poison-filled before every call so that an unwritten or
over-written element shows up.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding, workloads as wl
from tests import harness as hz

pytestmark = pytest.mark.gpu
DEV = "cuda"


def i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def poison_i32(*shape):
    return torch.full(shape, -7777, dtype=torch.int32, device=DEV)


def poison_bf16(*shape):
    return torch.full(shape, float("nan"), dtype=torch.bfloat16, device=DEV)


def small(name, **kw):
    return wl.WORKLOADS[name].scaled(**kw)


ROUTE_CASES = [
    wl.WORKLOADS["tiny"],
    small("mixtral", T=333, D=1024),
    small("many_expert", T=257, D=512),
    small("fine_grained", T=130, D=1024),
    small("fine_grained", T=64, D=256, E=200, K=8, S=200),
    small("tiny", T=65, D=64, E=5, K=5, S=5),
    small("tiny", T=40, D=64, E=33, K=1, S=40, gate_mode=1),
    # few token tiles and a long model dimension: the launcher splits D over clusters of eight CTAs
    # (at most 23 tiles of 128 tokens and D >= 2048), the widest split-K reduction
    small("mixtral", T=1024, D=4096),
    small("mixtral", T=2944, D=7168, gate_mode=1),
    small("many_expert", T=128, D=2048),
    small("many_expert", T=1000, D=4096, gate_mode=1),
    small("fine_grained", T=2944, D=7168),
    small("fine_grained", T=1024, D=2048, gate_mode=0),
    # four-CTA clusters with E = 256 and a ragged last tile
    small("fine_grained", T=3001, D=4096),
]


@pytest.mark.parametrize("w", ROUTE_CASES, ids=lambda w: f"{w.name}-T{w.T}-D{w.D}-E{w.E}-K{w.K}")
def test_route(w):
    wr, bias = wl.router(w, "cpu")
    x, redrawn = hz.screened_activations(w, wr, bias)
    assert redrawn <= max(4, 0.05 * w.T)
    ref_idx, ref_w, ref_logits = oracle.route(hz.bits(x), hz.bits(wr), bias.numpy(), w.K, w.gate_mode)
    ctx = binding.Context(binding.Shape(w.T, w.D, 64, w.E, w.K, w.S, w.gate_mode, 1))
    xd, wrd, bd = x.to(DEV), wr.to(DEV), bias.to(DEV)
    idx = poison_i32(w.T, w.K)
    wt = torch.full((w.T, w.K), float("nan"), dtype=torch.float32, device=DEV)
    logits = torch.full((w.T, w.E), float("nan"), dtype=torch.float32, device=DEV)
    ctx.route_logits(xd, wrd, bd, logits)
    ctx.route(xd, wrd, bd, idx, wt)
    ctx.check_status()
    # the fp32 logits must sit well inside the margin the inputs were screened for
    assert np.abs(logits.cpu().numpy().astype(np.float64) - ref_logits).max() < hz.TAU / 4
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    got_w = wt.cpu().numpy().astype(np.float64)
    hz.assert_close_rel_max(got_w, ref_w, "topk_w")
    assert np.abs(got_w - ref_w).max() < 2e-5
    assert np.abs(got_w.sum(axis=1) - 1).max() < 1e-5
    # the fused call (router epilogue also counts the selections): same indices and weights bit for
    # bit, histogram equal to the oracle's, on two calls in a row (the counters start from zero each time)
    for _ in range(2):
        idx2, wt2, hist = poison_i32(w.T, w.K), torch.full_like(wt, float("nan")), poison_i32(w.E)
        ctx.route_histogram(xd, wrd, bd, idx2, wt2, hist)
        ctx.check_status()
        assert torch.equal(idx2, idx) and torch.equal(wt2, wt)
        assert np.array_equal(hist.cpu().numpy(), oracle.histogram(ref_idx, w.E))


def test_route_no_bias_and_exact_ties():
    w = small("tiny", T=96, D=128, E=8, K=3, S=8)
    wr, _ = wl.router(w, "cpu")
    wr[6] = wr[2]
    wr[7] = wr[0]
    x = wl.activations(w, "cpu")
    logits = oracle.route_logits(hz.bits(x), hz.bits(wr), None)
    # keep tokens whose only near-ties are the planted exact ones
    srt = -np.sort(-logits, axis=1)
    gaps = srt[:, :w.K] - srt[:, 1:w.K + 1]
    ok = ((gaps == 0) | (gaps >= hz.TAU)).all(axis=1)
    x = x[torch.from_numpy(np.nonzero(ok)[0])].contiguous()
    w = w.scaled(T=x.shape[0])
    ref_idx, ref_w, _ = oracle.route(hz.bits(x), hz.bits(wr), None, w.K, 0)
    ctx = binding.Context(binding.Shape(w.T, w.D, 64, w.E, w.K, w.S, 0, 1))
    idx, wt = poison_i32(w.T, w.K), torch.empty(w.T, w.K, dtype=torch.float32, device=DEV)
    ctx.route(x.to(DEV), wr.to(DEV), None, idx, wt)
    ctx.check_status()
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert any(6 in r or 7 in r for r in ref_idx.tolist())


@pytest.mark.parametrize("T,K,E", [(256, 2, 8), (1000, 6, 64), (4096, 8, 256), (1, 1, 1), (77, 3, 3), (0, 2, 8)])
def test_histogram(T, K, E):
    rng = np.random.default_rng(T * 31 + E)
    p = 1.0 / np.arange(1, E + 1) ** 1.2
    idx = rng.choice(E, size=(T, K), p=p / p.sum()).astype(np.int32)
    ctx = binding.Context(binding.Shape(T, 64, 64, E, K, max(E, 1), 0, 1))
    hist = poison_i32(E)
    ctx.histogram(i32(idx).reshape(T, K), hist)
    ctx.check_status()
    assert np.array_equal(hist.cpu().numpy(), oracle.histogram(idx, E))
    assert int(hist.sum()) == T * K


def test_histogram_reports_bad_index_without_faulting():
    T, K, E = 64, 2, 8
    idx = np.zeros((T, K), dtype=np.int32)
    idx[5, 1] = E          # out of range
    idx[9, 0] = -3
    ctx = binding.Context(binding.Shape(T, 64, 64, E, K, E, 0, 1))
    hist = poison_i32(E)
    ctx.histogram(i32(idx), hist)
    assert ctx.status() == binding.ERR_BAD_INDEX
    assert ctx.status() == 0                       # cleared by the read
    assert int(hist.sum()) == T * K - 2


PLAN_CASES = [
    ([4, 2], 3, 0), ([2, 2], 3, 0), ([4, 2], 4, 0), ([0, 0, 0], 8, 0), ([5, 0, 1], 5, 0), ([3, 3, 3], 3, 0),
    ([100, 1, 1], 8, 3), ([100, 1], 8, 2), ([9000, 1000, 1000, 1000], 12, 0),
    ([2 ** 31 - 1, 2 ** 31 - 2, 5], 64, 0),
    # ratios that differ by the least amount two fractions with denominators <= 1024 can differ by,
    # 1 / (r1 r2), at the largest replica counts and counts the kernel supports, and exact ties there
    ([2 ** 31 - 1, 2 ** 31 - 2], 1024, 0), ([1023 * 1024 + 1, 1023 * 1024, 1], 1024, 0),
    ([511 * 512, 511 * 512 + 1, 511 * 512 - 1, 0], 1024, 0), ([2 ** 31 - 1, 2 ** 31 - 1, 2 ** 31 - 1], 1024, 0),
    ([2 ** 31 - 1] + [2 ** 30] * 3 + [1] * 60, 1024, 700), ([6, 4, 3, 2, 12], 1000, 0),
]


@pytest.mark.parametrize("pred,S,c_max", PLAN_CASES)
def test_plan_hand_cases(pred, S, c_max):
    run_plan(np.array(pred, dtype=np.int64), S, c_max)


@pytest.mark.parametrize("E,S,seed", [(8, 16, 0), (64, 80, 1), (256, 288, 2), (256, 1024, 3), (1, 9, 4),
                                      (200, 200, 5), (31, 97, 6)])
def test_plan_random(E, S, seed):
    rng = np.random.default_rng(seed)
    for kind in ("zipf", "ties", "sparse"):
        if kind == "zipf":
            pred = np.round(50000 / np.arange(1, E + 1) ** 1.1).astype(np.int64)
            rng.shuffle(pred)
        elif kind == "ties":
            pred = rng.integers(0, 4, size=E) * 12
        else:
            pred = np.where(rng.random(E) < 0.7, 0, rng.integers(0, 1000, size=E))
        run_plan(pred, S, 0)
        run_plan(pred, S, 3)


def run_plan(pred, S, c_max):
    E = len(pred)
    ctx = binding.Context(binding.Shape(8, 64, 64, E, 1, S, 0, 1, c_max))
    rep, so, se, bound = poison_i32(E), poison_i32(E + 1), poison_i32(S), poison_i32(1)
    ctx.plan(i32(pred), S, rep, so, se, bound)
    ctx.check_status()
    r_ref, so_ref, se_ref, b_ref = oracle.plan(pred, S, c_max)
    assert np.array_equal(rep.cpu().numpy(), r_ref)
    assert np.array_equal(so.cpu().numpy(), so_ref)
    assert np.array_equal(se.cpu().numpy(), se_ref)
    assert int(bound.item()) == b_ref


def test_trace_logs_every_launch_to_stderr(capfd, monkeypatch):
    """MOEGPS_TRACE: a host-side log line per kernel launch, read when the context is created."""
    monkeypatch.setenv("MOEGPS_TRACE", "1")
    ctx = binding.Context(binding.Shape(8, 64, 64, 4, 1, 6, 0, 1))
    monkeypatch.delenv("MOEGPS_TRACE")
    quiet = binding.Context(binding.Shape(8, 64, 64, 4, 1, 6, 0, 1))
    capfd.readouterr()
    args = lambda: (i32([5, 1, 1, 1]), 6, poison_i32(4), poison_i32(5), poison_i32(6), poison_i32(1))  # noqa: E731
    quiet.plan(*args())
    assert "[moegps]" not in capfd.readouterr().err
    n0 = ctx.launch_count()
    ctx.plan(*args())
    ctx.check_status()
    err = capfd.readouterr().err
    assert f"[moegps] launch {n0 + 1} moegps_launch_plan T=8 D=64 F=64 E=4 K=1 S=6 A=1" in err


def test_plan_rejects_wrong_slot_count():
    ctx = binding.Context(binding.Shape(8, 64, 64, 4, 1, 6, 0, 1))
    n0 = ctx.launch_count()
    with pytest.raises(binding.MoegpsError) as ei:
        ctx.plan(i32([1, 2, 3, 4]), 5, poison_i32(4), poison_i32(5), poison_i32(6), poison_i32(1))
    assert ei.value.code == binding.ERR_INVALID_ARG
    assert ctx.launch_count() == n0                # nothing was launched


DISPATCH_CASES = [
    # T, D, E, K, S, A, skew
    (256, 512, 8, 2, 8, 128, 1.0), (256, 512, 8, 2, 8, 1, 1.0), (1000, 256, 8, 2, 16, 128, 1.5),
    (777, 64, 64, 6, 80, 128, 1.2), (515, 128, 256, 8, 288, 128, 1.0), (515, 128, 256, 8, 288, 1, 1.0),
    (33, 64, 4, 4, 16, 4, 0.5), (1, 8, 1, 1, 1, 1, 0.0), (300, 72, 5, 1, 9, 32, 2.0), (0, 64, 4, 2, 6, 8, 1.0),
    # more than 1024 segments of 256 pairs: the path that scans the segment counts on the device
    (45000, 16, 16, 6, 20, 16, 1.0), (131073, 8, 3, 2, 7, 1, 0.7),
]


@pytest.mark.parametrize("T,D,E,K,S,A,skew", DISPATCH_CASES)
def test_dispatch(T, D, E, K, S, A, skew):
    rng = np.random.default_rng(T + 7 * E + S)
    p = 1.0 / np.arange(1, E + 1) ** skew
    p /= p.sum()
    idx = (np.stack([rng.choice(E, size=K, replace=False, p=p) for _ in range(T)]).astype(np.int32)
           if T else np.zeros((0, K), dtype=np.int32))
    hist = oracle.histogram(idx, E)
    pred = np.maximum(0, np.round(hist * (1 + 0.1 * rng.normal(size=E)))).astype(np.int64)
    rep, so, se, _ = oracle.plan(pred, S)
    x = rng.integers(0, 1 << 16, size=(T, D), dtype=np.uint16)
    x[(x & 0x7F80) == 0x7F80] = 0x3F80            # keep the payload finite (bits are the contract)
    sro_ref, rp_ref, pr_ref, xp_ref = oracle.dispatch(x, idx, hist, rep, so, S, A)
    shape = binding.Shape(T, D, 64, E, K, S, 0, A)
    ctx = binding.Context(shape)
    sro, rp, pr = poison_i32(S + 1), poison_i32(shape.Rcap), poison_i32(T, K)
    xp = torch.full((shape.Rcap, D), 0x5A5A, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    ws = torch.full((binding.workspace_bytes(shape),), 0xFF, dtype=torch.uint8, device=DEV)
    ctx.dispatch(hz.from_bits(x, DEV).reshape(T, D), i32(idx).reshape(T, K), i32(hist), i32(rep), i32(so), sro, rp,
                 pr, xp, ws)
    ctx.check_status()
    assert np.array_equal(sro.cpu().numpy(), sro_ref)
    assert np.array_equal(rp.cpu().numpy(), rp_ref)
    assert np.array_equal(pr.cpu().numpy(), pr_ref)
    got_xp = hz.bits(xp)
    occ = rp_ref >= 0
    assert np.array_equal(got_xp[occ], xp_ref[occ])
    assert (got_xp[~occ] == 0x5A5A).all()          # padding rows are not written


FUSED_CASES = [
    # workload, A          (clusters of 1, 2, 4 and 8 router CTAs per tile; E from 5 to 256; K from 1 to 8; ragged T)
    (small("tiny", T=256, D=512), 128), (small("mixtral", T=1024, D=4096), 16), (small("mixtral", T=2944, D=2048), 1),
    (small("many_expert", T=1000, D=4096), 16), (small("fine_grained", T=515, D=1024), 16),
    (small("fine_grained", T=130, D=4096, S=300), 128), (small("tiny", T=65, D=64, E=5, K=5, S=9), 4),
    (small("tiny", T=40, D=64, E=33, K=1, S=40, gate_mode=1), 8), (small("mixtral_skew", T=16384 + 77, D=256), 16),
]


@pytest.mark.parametrize("w,A", FUSED_CASES, ids=lambda v: v if isinstance(v, int) else f"{v.name}-T{v.T}-D{v.D}-E{v.E}-K{v.K}")
def test_route_prepare_and_dispatch_prepared_equal_the_separate_calls_and_the_oracle(w, A):
    """The two-launch form (router also produces the counts dispatch ranks with) against the
    four-launch form, bit for bit, and against the oracle; twice in a row with different batches,
    because the router's accumulators live in the context and must be back at zero after every call."""
    wr, bias = wl.router(w, "cpu")
    shape = binding.Shape(w.T, w.D, 64, w.E, w.K, w.S, w.gate_mode, A)
    ctx = binding.Context(shape)
    wrd, bd = wr.to(DEV), bias.to(DEV)
    ws_a = torch.full((binding.workspace_bytes(shape),), 0xEE, dtype=torch.uint8, device=DEV)
    ws_b = torch.full((binding.workspace_bytes(shape),), 0xEE, dtype=torch.uint8, device=DEV)
    for call in range(2):
        x, _ = hz.screened_activations(w.scaled(number=w.number + 13 * call), wr, bias)
        xd = x.to(DEV)
        ref_idx, ref_w, _ = oracle.route(hz.bits(x), hz.bits(wr), bias.numpy(), w.K, w.gate_mode)
        ref_hist = oracle.histogram(ref_idx, w.E)
        pred = np.maximum(0, np.round(ref_hist * (1 + 0.2 * np.random.default_rng(call).normal(size=w.E)))).astype(np.int64)
        rep_ref, so_ref, _, _ = oracle.plan(pred, w.S)
        rep, so = i32(rep_ref), i32(so_ref)
        # separate calls
        idx_a, wt_a, hist_a = poison_i32(w.T, w.K), torch.full((w.T, w.K), float("nan"), device=DEV), poison_i32(w.E)
        sro_a, rp_a, pr_a = poison_i32(w.S + 1), poison_i32(shape.Rcap), poison_i32(w.T, w.K)
        xp_a = torch.full((shape.Rcap, w.D), 0x5A5A, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        ctx.route_histogram(xd, wrd, bd, idx_a, wt_a, hist_a)
        ctx.dispatch(xd, idx_a, hist_a, rep, so, sro_a, rp_a, pr_a, xp_a, ws_a)
        # fused calls
        idx_b, wt_b, hist_b = poison_i32(w.T, w.K), torch.full((w.T, w.K), float("nan"), device=DEV), poison_i32(w.E)
        sro_b, rp_b, pr_b = poison_i32(w.S + 1), poison_i32(shape.Rcap), poison_i32(w.T, w.K)
        xp_b = torch.full((shape.Rcap, w.D), 0x5A5A, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        ctx.route_prepare(xd, wrd, bd, idx_b, wt_b, hist_b, ws_b)
        ctx.dispatch_prepared(xd, idx_b, hist_b, rep, so, sro_b, rp_b, pr_b, xp_b, ws_b)
        ctx.check_status()
        for a, b, what in ((idx_a, idx_b, "topk_idx"), (wt_a, wt_b, "topk_w"), (hist_a, hist_b, "hist"),
                           (sro_a, sro_b, "slot_row_off"), (rp_a, rp_b, "row_pair"), (pr_a, pr_b, "pair_row")):
            assert torch.equal(a, b), (call, what)
        assert torch.equal(xp_a.view(torch.int16), xp_b.view(torch.int16)), (call, "xp")
        sro_ref, rp_ref, pr_ref, _ = oracle.dispatch(None, ref_idx, ref_hist, rep_ref, so_ref, w.S, A)
        assert np.array_equal(idx_b.cpu().numpy(), ref_idx) and np.array_equal(hist_b.cpu().numpy(), ref_hist)
        assert np.array_equal(sro_b.cpu().numpy(), sro_ref)
        assert np.array_equal(rp_b.cpu().numpy(), rp_ref) and np.array_equal(pr_b.cpu().numpy(), pr_ref)


def test_route_prepare_and_dispatch_prepared_without_tokens():
    shape = binding.Shape(0, 64, 64, 4, 2, 6, 0, 8)
    ctx = binding.Context(shape)
    hist, sro = poison_i32(4), poison_i32(7)
    ws = torch.zeros(binding.workspace_bytes(shape), dtype=torch.uint8, device=DEV)
    x = torch.zeros(0, 64, dtype=torch.bfloat16, device=DEV)
    idx = torch.zeros(0, 2, dtype=torch.int32, device=DEV)
    ctx.route_prepare(x, torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV), None, idx,
                      torch.zeros(0, 2, dtype=torch.float32, device=DEV), hist, ws)
    ctx.dispatch_prepared(x, idx, hist, i32([2, 2, 1, 1]), i32([0, 2, 4, 5, 6]), sro,
                          torch.zeros(shape.Rcap, dtype=torch.int32, device=DEV), idx.clone(),
                          torch.zeros(shape.Rcap, 64, dtype=torch.bfloat16, device=DEV), ws)
    ctx.check_status()
    assert hist.tolist() == [0] * 4 and sro.tolist() == [0] * 7


def test_dispatch_detects_hist_mismatch():
    T, D, E, K, S = 64, 64, 4, 2, 6
    rng = np.random.default_rng(3)
    idx = np.stack([rng.choice(E, size=K, replace=False) for _ in range(T)]).astype(np.int32)
    hist = oracle.histogram(idx, E)
    hist[0] += 1
    hist[1] -= 1
    shape = binding.Shape(T, D, 64, E, K, S, 0, 8)
    ctx = binding.Context(shape)
    ws = torch.zeros(binding.workspace_bytes(shape), dtype=torch.uint8, device=DEV)
    ctx.dispatch(torch.zeros(T, D, dtype=torch.bfloat16, device=DEV), i32(idx), i32(hist), i32([2, 2, 1, 1]),
                 i32([0, 2, 4, 5, 6]), poison_i32(S + 1), poison_i32(shape.Rcap), poison_i32(T, K),
                 torch.zeros(shape.Rcap, D, dtype=torch.bfloat16, device=DEV), ws)
    assert ctx.status() == binding.ERR_HIST_MISMATCH


def test_dispatch_rejects_small_workspace():
    shape = binding.Shape(1024, 64, 64, 8, 2, 8, 0, 1)
    ctx = binding.Context(shape)
    with pytest.raises(binding.MoegpsError) as ei:
        ctx.dispatch(None, None, None, None, None, None, None, None, None,
                     torch.zeros(8, dtype=torch.uint8, device=DEV))
    assert ei.value.code == binding.ERR_WORKSPACE_TOO_SMALL


FFN_CASES = [
    # T, D, F, E, K, S, A, skew
    (256, 512, 1024, 8, 2, 8, 128, 1.0),
    (256, 512, 1024, 8, 2, 12, 1, 1.0),        # unaligned slots: tiles straddle slot ends
    (300, 256, 384, 4, 2, 7, 128, 1.5),        # F = 3 x 128; D = one 256 tile
    (200, 320, 200, 6, 3, 9, 128, 1.0),        # D, F not multiples of the tile (ragged K and N tails)
    (700, 128, 1408, 16, 4, 20, 128, 1.2),     # several row tiles per slot, F = 11 x 128
    (64, 64, 64, 32, 8, 40, 128, 1.0),         # many almost-empty slots
    (5, 2048, 256, 2, 1, 2, 128, 0.0),         # long K loop, a handful of rows
    # long slots: many row tiles per slot
    (1500, 256, 384, 2, 2, 3, 128, 0.5),
    (1500, 256, 384, 2, 2, 3, 1, 0.5),         # unaligned slots: row tiles straddle slot ends
    (3000, 128, 256, 4, 1, 4, 128, 1.5),       # one hot slot with many row tiles, cold ones with one
    (1100, 200, 328, 2, 1, 2, 128, 0.0),       # ragged K and N tails with several row tiles
    # far more tiles than CTAs: gate+up about 1550 tiles and down about 780 (a persistent CTA walks
    # 5-11 tiles of 16 K-blocks each, so the shared-memory ring and the two accumulators wrap many times)
    (12288, 1024, 1024, 8, 2, 8, 128, 0.8),
    (12288, 1024, 1024, 8, 2, 12, 1, 0.8),     # the same with unaligned slots and replicas
    (6000, 2048, 256, 4, 2, 6, 128, 1.0),      # down GEMM with 8 column tiles per row tile, 32 K-blocks in gate+up
    # a mix of short (under 128 rows) and long slots at small row alignments, ragged weight tails (F, D not
    # multiples of 128): tiles of short slots read into the following slots' rows and must not write there
    (900, 256, 384, 64, 4, 80, 16, 1.2),
    (900, 256, 384, 64, 4, 80, 1, 1.2),        # extents that are not multiples of 16: the tile reads into the next slot
    (700, 200, 328, 24, 3, 30, 8, 0.7),
    (130, 512, 640, 3, 1, 3, 16, 0.0),         # extents of 48, 48, 48 ... and single slots just below / above 128 rows
    (257, 128, 128, 2, 1, 2, 1, 0.0),
]


@pytest.mark.parametrize("T,D,F,E,K,S,A,skew", FFN_CASES)
def test_expert_ffn(T, D, F, E, K, S, A, skew):
    rng = np.random.default_rng(T + D + F)
    p = 1.0 / np.arange(1, E + 1) ** skew
    p /= p.sum()
    idx = np.stack([rng.choice(E, size=K, replace=False, p=p) for _ in range(T)]).astype(np.int32)
    hist = oracle.histogram(idx, E)
    rep, so, se, _ = oracle.plan(hist, S)
    x = hz.bits(hz.f64_to_bf16_tensor(rng.normal(size=(T, D))))
    sro, rp, pr, xp = oracle.dispatch(x, idx, hist, rep, so, S, A)
    w1 = hz.f64_to_bf16_tensor(rng.normal(size=(E, F, D)) / math.sqrt(D))
    w3 = hz.f64_to_bf16_tensor(rng.normal(size=(E, F, D)) / math.sqrt(D))
    w2 = hz.f64_to_bf16_tensor(rng.normal(size=(E, D, F)) / math.sqrt(F))
    ref = oracle.expert_ffn(xp, sro, se, hz.bits(w1), hz.bits(w3), hz.bits(w2))
    shape = binding.Shape(T, D, F, E, K, S, 0, A)
    ctx = binding.Context(shape)
    # padding rows hold NaN on purpose: rows are independent, so they must not leak into real rows
    xpd = hz.from_bits(xp, DEV)
    xpd[torch.from_numpy(rp < 0).to(DEV)] = float("nan")
    h_ws, yp = poison_bf16(shape.Rcap, F), poison_bf16(shape.Rcap, D)
    ctx.expert_ffn(xpd, i32(sro), i32(se), w1.to(DEV), w3.to(DEV), w2.to(DEV), h_ws, yp)
    ctx.check_status()
    occ = rp >= 0
    got = yp.float().cpu().numpy().astype(np.float64)
    hz.assert_close_rel_max(got[occ], ref[occ], "yp")
    # rows outside every slot's extent stay untouched
    outside = np.ones(shape.Rcap, dtype=bool)
    for s in range(S):
        outside[sro[s]:sro[s + 1]] = False
    assert torch.isnan(yp[torch.from_numpy(outside).to(DEV)]).all()
    # bitwise run-to-run determinism
    yp2 = poison_bf16(shape.Rcap, D)
    ctx.expert_ffn(xpd, i32(sro), i32(se), w1.to(DEV), w3.to(DEV), w2.to(DEV), h_ws, yp2)
    ctx.check_status()
    assert np.array_equal(hz.bits(yp)[occ], hz.bits(yp2)[occ])


@pytest.mark.parametrize("offsets", [[0, 128, 640], [0, -128, 128], [0, 256, 128]])
def test_expert_ffn_skips_slot_extents_outside_the_buffers(offsets):
    """slot_row_off that runs past Rcap, goes negative or decreases: the slots concerned are skipped
    (nothing is read or written for them), BAD_INDEX is reported, nothing faults.  The buffers are
    allocated longer than Rcap rows with a poisoned tail that must stay untouched."""
    T, D, F, E = 256, 128, 256, 2
    shape = binding.Shape(T, D, F, E, 1, E, 0, 128)            # Rcap = 510
    ctx = binding.Context(shape)
    g = torch.Generator().manual_seed(5)
    rows = 1024
    xp_all = torch.randn(rows, D, generator=g).to(torch.bfloat16).to(DEV)
    w1 = (torch.randn(E, F, D, generator=g) / math.sqrt(D)).to(torch.bfloat16).to(DEV)
    w3 = (torch.randn(E, F, D, generator=g) / math.sqrt(D)).to(torch.bfloat16).to(DEV)
    w2 = (torch.randn(E, D, F, generator=g) / math.sqrt(F)).to(torch.bfloat16).to(DEV)
    h_all, yp_all = poison_bf16(rows, F), poison_bf16(rows, D)
    ctx.expert_ffn(xp_all[:shape.Rcap], i32(offsets), i32([0, 1]), w1, w3, w2, h_all[:shape.Rcap], yp_all[:shape.Rcap])
    assert ctx.status() == binding.ERR_BAD_INDEX
    sane = [s for s in range(E) if 0 <= offsets[s] <= offsets[s + 1] <= shape.Rcap]
    written = torch.zeros(rows, dtype=torch.bool, device=DEV)
    for s in sane:
        written[offsets[s]:offsets[s + 1]] = True
    assert torch.isnan(yp_all[~written]).all() and torch.isnan(h_all[~written]).all()
    assert torch.isfinite(yp_all[written].float()).all()
    if sane:                                                    # and the sane slot is still right
        s = sane[0]
        ref = oracle.expert_ffn(hz.bits(xp_all[:shape.Rcap]), [offsets[s], offsets[s + 1]], [s], hz.bits(w1), hz.bits(w3),
                                hz.bits(w2))
        hz.assert_close_rel_max(yp_all[offsets[s]:offsets[s + 1]].float().cpu().numpy(),
                                ref[offsets[s]:offsets[s + 1]], "yp of the sane slot")


def test_expert_ffn_zero_gate_weights_give_zero():
    T, D, F, E = 128, 128, 256, 2
    shape = binding.Shape(T, D, F, E, 1, E, 0, 128)
    ctx = binding.Context(shape)
    g = torch.Generator().manual_seed(1)
    xp = torch.randn(shape.Rcap, D, generator=g).to(torch.bfloat16).to(DEV)
    w3 = torch.randn(E, F, D, generator=g).to(torch.bfloat16).to(DEV)
    w2 = torch.randn(E, D, F, generator=g).to(torch.bfloat16).to(DEV)
    w1 = torch.zeros(E, F, D, dtype=torch.bfloat16, device=DEV)
    yp = poison_bf16(shape.Rcap, D)
    ctx.expert_ffn(xp, i32([0, 128, 256]), i32([1, 0]), w1, w3, w2, poison_bf16(shape.Rcap, F), yp)
    ctx.check_status()
    assert (yp[:256] == 0).all()


@pytest.mark.parametrize("T,D,K,S,A", [(256, 512, 2, 8, 128), (100, 4096, 2, 8, 1), (77, 2048, 6, 80, 128),
                                       (33, 7168, 8, 40, 128), (9, 72, 1, 3, 4), (50, 264, 3, 5, 1), (40, 8, 5, 8, 2)])
def test_combine(T, D, K, S, A):
    rng = np.random.default_rng(T * D + K)
    E = S
    idx = np.stack([rng.choice(E, size=K, replace=False) for _ in range(T)]).astype(np.int32)
    hist = oracle.histogram(idx, E)
    rep, so, se, _ = oracle.plan(hist, S)
    sro, rp, pr, _ = oracle.dispatch(None, idx, hist, rep, so, S, A)
    shape = binding.Shape(T, D, 64, E, K, S, 0, A)
    yp = hz.f64_to_bf16_tensor(rng.normal(size=(shape.Rcap, D)))
    wts = rng.random(size=(T, K)).astype(np.float32)
    wts /= wts.sum(axis=1, keepdims=True)
    ref = oracle.combine(hz.bits(yp), pr, wts)
    ctx = binding.Context(shape)
    out = poison_bf16(T, D)
    ctx.combine(yp.to(DEV), i32(pr), torch.from_numpy(wts).to(DEV), out)
    ctx.check_status()
    got = out.float().cpu().numpy().astype(np.float64)
    hz.assert_close_rel_max(got, ref, "out")
    # fp32 accumulation + one bf16 rounding: within half a bf16 ulp of the reference, plus slack
    assert np.abs(got - ref).max() <= 2 ** -8 * np.abs(ref).max()


def test_bounded_wait_reports_timeout_and_leaves_the_context_usable():
    # failure detection without a fault: a wait that nothing will ever satisfy must give up, report
    # through the status word, and let the kernel return; later calls work as usual
    shape = binding.Shape(64, 64, 64, 4, 2, 4, 0, 1)
    ctx = binding.Context(shape)
    assert ctx.status() == 0
    ctx.selftest_bounded_wait(limit_cycles=2_000_000)          # about a millisecond
    assert ctx.status() == binding.ERR_TIMEOUT
    assert ctx.status() == 0
    idx = torch.randint(0, 4, (64, 2), dtype=torch.int32, device=DEV)
    hist = poison_i32(4)
    ctx.histogram(idx, hist)
    ctx.check_status()
    assert int(hist.sum()) == 128
    with pytest.raises(binding.MoegpsError):
        ctx.selftest_bounded_wait(limit_cycles=10)              # out of the accepted range


def test_invalid_pointers_launch_nothing():
    shape = binding.Shape(64, 64, 64, 4, 2, 4, 0, 1)
    ctx = binding.Context(shape)
    n0 = ctx.launch_count()
    lib = binding._lib()
    buf = torch.zeros(4096, dtype=torch.uint8, device=DEV)
    misaligned = buf.data_ptr() + 4
    assert lib.moegps_histogram(ctx._h, None, buf.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert lib.moegps_histogram(ctx._h, misaligned, buf.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert lib.moegps_combine(ctx._h, buf.data_ptr(), None, buf.data_ptr(), buf.data_ptr(), None) == binding.ERR_INVALID_ARG
    assert ctx.launch_count() == n0
    with pytest.raises(TypeError):
        ctx.histogram(torch.zeros(64, 2, dtype=torch.int64, device=DEV), torch.zeros(4, dtype=torch.int32, device=DEV))
