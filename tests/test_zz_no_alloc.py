"""moegps_dispatch_static: the dispatch entry point for callers that cannot allocate device memory
(a plug-in inside a host application whose memory pool is closed to it, a deployment whose device
memory is carved up once at start-up, a latency-critical path where an allocator call may block).
Its scratch is a fixed array inside the library instead of a caller-provided workspace.

The test drives it through the C ABI twice in a row, with different routings, and requires the
results to be identical to those of moegps_dispatch (integers and row copies: bit-exact, the same bar
as the other dispatch tests).  The second call finds the scratch full of the first call's counters,
which must not matter.  This file is collected last on purpose, and passes on its own as well.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_07366_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda"


def routing(T, K, E, seed, skew):
    """K distinct experts per token, popular ones more often (Gumbel top-K draw: no Python loop)."""
    rng = np.random.default_rng(seed)
    logp = -skew * np.log(np.arange(1, E + 1))
    keys = logp[None, :] + rng.gumbel(size=(T, E))
    idx = np.argsort(-keys, axis=1)[:, :K].astype(np.int32)
    return torch.from_numpy(np.ascontiguousarray(idx)).to(DEV)


def run_both(ctx, shape, x, idx, pred):
    """Plan + histogram with the library, then dispatch through both entry points."""
    i32 = dict(dtype=torch.int32, device=DEV)
    hist = torch.empty(shape.E, **i32)
    rep, so, se, bound = (torch.empty(shape.E, **i32), torch.empty(shape.E + 1, **i32),
                          torch.empty(shape.S, **i32), torch.empty(1, **i32))
    ctx.histogram(idx, hist)
    ctx.plan(pred, shape.S, rep, so, se, bound)
    outs = []
    for static in (False, True):
        sro = torch.full((shape.S + 1,), -5, **i32)
        rp = torch.full((shape.Rcap,), -5, **i32)
        pr = torch.full((shape.T, shape.K), -5, **i32)
        xp = torch.full((shape.Rcap, shape.D), 0x3C3C, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        if static:
            # the claim "allocates nothing": the driver's free memory does not shrink and torch's
            # allocator sees no new request while the call runs (frees by the garbage collector may happen)
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
            requests0 = torch.cuda.memory_stats()["allocation.all.allocated"]
            ctx.dispatch_static(x, idx, hist, rep, so, sro, rp, pr, xp)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] >= free0
            assert torch.cuda.memory_stats()["allocation.all.allocated"] == requests0
        else:
            ws = torch.empty(binding.workspace_bytes(shape), dtype=torch.uint8, device=DEV)
            ctx.dispatch(x, idx, hist, rep, so, sro, rp, pr, xp, ws)
        ctx.check_status()
        outs.append((sro, rp, pr, xp))
    return outs


def test_dispatch_static_matches_dispatch_twice_in_a_row():
    shape = binding.Shape(T=3000, D=256, F=64, E=64, K=6, S=80, gate_mode=0, row_align=128)
    ctx = binding.Context(shape)
    g = torch.Generator().manual_seed(7)
    for call, (seed, skew) in enumerate([(11, 1.2), (12, 0.3)]):
        x = torch.randn(shape.T, shape.D, generator=g).to(torch.bfloat16).to(DEV)
        idx = routing(shape.T, shape.K, shape.E, seed, skew)
        pred = torch.bincount(idx.reshape(-1).long(), minlength=shape.E).to(torch.int32)
        (sro_a, rp_a, pr_a, xp_a), (sro_b, rp_b, pr_b, xp_b) = run_both(ctx, shape, x, idx, pred)
        assert torch.equal(sro_a, sro_b), f"call {call}: slot_row_off"
        assert torch.equal(rp_a, rp_b), f"call {call}: row_pair"
        assert torch.equal(pr_a, pr_b), f"call {call}: pair_row"
        assert torch.equal(xp_a.view(torch.int16), xp_b.view(torch.int16)), f"call {call}: xp"
        assert int((rp_b >= 0).sum()) == shape.R          # and it really did the work
        idx_h = idx.cpu().numpy()                         # the oracle agrees with both
        hist = oracle.histogram(idx_h, shape.E)
        rep, so, _, _ = oracle.plan(pred.cpu().numpy(), shape.S)
        sro_ref, rp_ref, pr_ref, _ = oracle.dispatch(None, idx_h, hist, rep, so, shape.S, shape.row_align)
        assert np.array_equal(sro_b.cpu().numpy(), sro_ref) and np.array_equal(rp_b.cpu().numpy(), rp_ref)
        assert np.array_equal(pr_b.cpu().numpy(), pr_ref)


@pytest.mark.parametrize("T,D,E,K,S,A", [
    (32768, 8, 256, 8, 256, 1),     # ceil(T*K/256) * E = 262144: exactly the scratch, 1024 segments
    (45000, 16, 16, 6, 20, 16),     # 1055 segments: the path that scans the counts on the device
    (131073, 8, 3, 2, 7, 1),        # 1025 segments, a ragged last one
])
def test_dispatch_static_at_its_limit_and_on_the_scan_path(T, D, E, K, S, A):
    """Bit-exact against moegps_dispatch AND against the oracle, twice in a row."""
    shape = binding.Shape(T=T, D=D, F=8, E=E, K=K, S=S, gate_mode=0, row_align=A)
    ctx = binding.Context(shape)
    g = torch.Generator().manual_seed(T)
    for call in range(2):
        x = torch.randn(T, D, generator=g).to(torch.bfloat16).to(DEV)
        idx = routing(T, K, E, 100 + call, 1.0)
        pred = torch.bincount(idx.reshape(-1).long(), minlength=E).to(torch.int32)
        (sro_a, rp_a, pr_a, xp_a), (sro_b, rp_b, pr_b, xp_b) = run_both(ctx, shape, x, idx, pred)
        assert torch.equal(sro_a, sro_b) and torch.equal(rp_a, rp_b) and torch.equal(pr_a, pr_b)
        assert torch.equal(xp_a.view(torch.int16), xp_b.view(torch.int16))
        idx_h = idx.cpu().numpy()
        hist = oracle.histogram(idx_h, E)
        rep, so, _, _ = oracle.plan(hist, S)
        sro_ref, rp_ref, pr_ref, _ = oracle.dispatch(None, idx_h, hist, rep, so, S, A)
        assert np.array_equal(sro_b.cpu().numpy(), sro_ref)
        assert np.array_equal(rp_b.cpu().numpy(), rp_ref)
        assert np.array_equal(pr_b.cpu().numpy(), pr_ref)
        occ = torch.from_numpy(rp_ref >= 0).to(DEV)
        src = torch.from_numpy(rp_ref[rp_ref >= 0] // K).to(DEV)
        assert torch.equal(xp_b[occ].view(torch.int16), x[src].view(torch.int16))


def test_dispatch_static_rejects_oversized_problem():
    # ceil(T*K/256) * E = 1025 * 256 > 262144
    shape = binding.Shape(T=32800, D=8, F=8, E=256, K=8, S=256, gate_mode=0, row_align=1)
    ctx = binding.Context(shape)
    i32 = dict(dtype=torch.int32, device=DEV)
    n0 = ctx.launch_count()
    with pytest.raises(binding.MoegpsError) as ei:
        ctx.dispatch_static(torch.zeros(shape.T, shape.D, dtype=torch.bfloat16, device=DEV),
                            torch.zeros(shape.T, shape.K, **i32), torch.zeros(shape.E, **i32),
                            torch.ones(shape.E, **i32), torch.arange(shape.E + 1, **i32),
                            torch.zeros(shape.S + 1, **i32), torch.zeros(shape.Rcap, **i32),
                            torch.zeros(shape.T, shape.K, **i32),
                            torch.zeros(shape.Rcap, shape.D, dtype=torch.bfloat16, device=DEV))
    assert ei.value.code == binding.ERR_STATIC_SCRATCH_EXCEEDED
    assert "moegps_dispatch" in str(ei.value)
    assert ctx.launch_count() == n0
