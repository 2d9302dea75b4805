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
    ([100], [0], [1, 1, 1], 0), ([0, 0, 0], [2, 1, 0], [1, 1, 1], 0), ([2 ** 31 - 1, 5], [0, 1], [2, 2], 0),
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
    ctx = binding.Context(binding.Shape(8, 64, 64, 4, 1, 4, 0, 1))
    with pytest.raises(binding.MoegpsError) as ei:                                                # too many devices
        ctx.pack(i32([1] * 4), i32([0] * 4), i32([4] * 65), 65, torch.zeros(4, 65, dtype=torch.int32, device=DEV),
                 torch.zeros(4, 65, dtype=torch.int32, device=DEV), torch.zeros(65, dtype=torch.int32, device=DEV),
                 torch.zeros(1, dtype=torch.int32, device=DEV))
    assert ei.value.code == binding.ERR_UNSUPPORTED_SHAPE
