"""Pins for the CPU oracle: each test checks an oracle function against something other than
itself - a value the paper prints, a closed form, a textbook/library routine, an invariant, or a
brute-force search on tiny inputs."""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))
rng = np.random.default_rng(20250607)


def to_bf16_bits(a):
    t = torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------------------ number format
def test_bf16_decode_known_patterns():
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x3DCD, 0x7F7F, 0x8000], dtype=np.uint16)
    got = oracle.bf16_bits_to_f64(bits)
    want = [1.0, -2.0, 0.0, 0.10009765625, 3.3895313892515355e38, -0.0]
    assert got.tolist() == want
    assert math.copysign(1.0, got[-1]) == -1.0


def test_bf16_decode_matches_torch():
    bits = rng.integers(0, 1 << 16, size=4096, dtype=np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]          # finite values only
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64)
    assert np.array_equal(oracle.bf16_bits_to_f64(bits), t.numpy())


# ------------------------------------------------------------------------------ route
def brute_force_topk(logits_row, K):
    """Repeatedly extract the maximum; among equal values the lower index wins."""
    left = list(range(len(logits_row)))
    out = []
    for _ in range(K):
        best = left[0]
        for e in left[1:]:
            if logits_row[e] > logits_row[best]:
                best = e
        out.append(best)
        left.remove(best)
    return out


def test_route_logits_one_hot_closed_form():
    # X rows are unit vectors: logit[t, e] must be Wr[e, d_t] + b[e] (catches a transposed operand).
    T, D, E = 5, 7, 3
    d_of_t = [6, 0, 3, 3, 1]
    X = np.zeros((T, D))
    for t, d in enumerate(d_of_t):
        X[t, d] = 1.0
    Wr = oracle.bf16_bits_to_f64(to_bf16_bits(rng.normal(size=(E, D))))
    b = rng.normal(size=E).astype(np.float32)
    got = oracle.route_logits(to_bf16_bits(X), to_bf16_bits(Wr), b)
    for t, d in enumerate(d_of_t):
        for e in range(E):
            assert got[t, e] == Wr[e, d] + float(b[e])


@pytest.mark.parametrize("E,K,mode", [(8, 2, 0), (8, 8, 0), (16, 1, 0), (32, 6, 1), (5, 3, 1)])
def test_route_selection_brute_force(E, K, mode):
    T, D = 64, 24
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)) / math.sqrt(D))
    b = rng.normal(size=E).astype(np.float32)
    idx, w, logits = oracle.route(x, wr, b, K, mode)
    assert idx.shape == (T, K) and w.shape == (T, K) and idx.dtype == np.int32
    for t in range(T):
        assert idx[t].tolist() == brute_force_topk(logits[t], K)
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-12)
    assert (w > 0).all()


def test_route_full_softmax_when_k_equals_e():
    T, D, E = 16, 12, 6
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)))
    idx, w, logits = oracle.route(x, wr, None, E, 0)
    full = scipy.special.softmax(logits, axis=1)
    assert np.allclose(w, np.take_along_axis(full, idx.astype(np.int64), axis=1), rtol=1e-12)


def test_route_softmax_is_full_softmax_renormalised():
    T, D, E, K = 16, 12, 9, 3
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)))
    idx, w, logits = oracle.route(x, wr, None, K, 0)
    full = scipy.special.softmax(logits, axis=1)
    sel = np.take_along_axis(full, idx.astype(np.int64), axis=1)
    assert np.allclose(w, sel / sel.sum(axis=1, keepdims=True), rtol=1e-12)


def test_route_sigmoid_mode_ratios():
    T, D, E, K = 16, 12, 9, 4
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)))
    b = rng.normal(size=E).astype(np.float32)
    idx, w, logits = oracle.route(x, wr, b, K, 1)
    s = scipy.special.expit(np.take_along_axis(logits, idx.astype(np.int64), axis=1))
    assert np.allclose(w * s.sum(axis=1, keepdims=True), s, rtol=1e-12)
    # descending logits => descending weights in both modes
    assert (np.diff(w, axis=1) <= 0).all()


def test_route_k1_weight_is_one():
    x = to_bf16_bits(rng.normal(size=(8, 4)))
    wr = to_bf16_bits(rng.normal(size=(3, 4)))
    for mode in (0, 1):
        idx, w, logits = oracle.route(x, wr, None, 1, mode)
        assert np.array_equal(w, np.ones((8, 1)))
        assert np.array_equal(idx[:, 0], logits.argmax(axis=1))


def test_route_exact_ties_go_to_lower_index():
    T, D, E = 32, 16, 6
    wr = rng.normal(size=(E, D))
    wr[4] = wr[1]                       # experts 1 and 4 always tie exactly
    wr[5] = wr[0]                       # experts 0 and 5 too
    x = to_bf16_bits(rng.normal(size=(T, D)))
    idx, w, logits = oracle.route(x, to_bf16_bits(wr), None, 3, 0)
    for t in range(T):
        sel = idx[t].tolist()
        if 4 in sel:
            assert 1 in sel and sel.index(1) < sel.index(4)
        if 5 in sel:
            assert 0 in sel and sel.index(0) < sel.index(5)
    assert any(4 in idx[t] or 5 in idx[t] for t in range(T))


def test_route_expert_permutation_equivariance():
    T, D, E, K = 32, 16, 8, 3
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)))
    b = rng.normal(size=E).astype(np.float32)
    perm = rng.permutation(E)
    idx, w, _ = oracle.route(x, wr, b, K, 0)
    idx2, w2, _ = oracle.route(x, wr[perm], b[perm], K, 0)
    assert np.array_equal(perm[idx2], idx)
    assert np.allclose(w2, w, rtol=1e-12)


# ------------------------------------------------------------------------------ histogram / stats
def test_histogram_against_bincount_and_sum():
    T, K, E = 300, 3, 11
    idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
    h = oracle.histogram(idx, E)
    assert h.sum() == T * K
    assert np.array_equal(h, np.bincount(idx.reshape(-1), minlength=E))
    with pytest.raises(ValueError):
        oracle.histogram(np.array([[0, E]]), E)
    with pytest.raises(ValueError):
        oracle.histogram(np.array([[-1, 0]]), E)
    assert oracle.histogram(np.zeros((0, 2), dtype=np.int32), 4).tolist() == [0, 0, 0, 0]


def test_skewness_paper_example():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "skewness_example.txt"))
            if l.strip() and not l.startswith("#")]
    share, n_exp, want = float(rows[0][0]), int(rows[0][1]), float(rows[0][2])
    total = 1200
    top = int(round(share * total))
    rest = (total - top) // (n_exp - 1)
    hist = [top] + [rest] * (n_exp - 1)
    assert sum(hist) == total
    assert oracle.skewness(hist) == want
    assert oracle.skewness([7, 7, 7, 7, 7]) == 1.0


def test_p_hat_and_error_rate():
    h = np.array([6, 3, 1, 0])
    p = oracle.p_hat(h)
    assert p.tolist() == [0.6, 0.3, 0.1, 0.0] and abs(p.sum() - 1) < 1e-15
    assert oracle.error_rate(p, p) == 0.0
    # hand-worked: E = 4, estimate (1/2, 1/2, 0, 0) against the uniform truth: every expert is off
    # by 1/4 = one unit of 1/E, so the average is exactly 1.
    assert oracle.error_rate([0.5, 0.5, 0.0, 0.0], [0.25] * 4) == 1.0
    # one expert off by 0.1 up, another 0.1 down, E = 5: (0.1 + 0.1) / 5 / (1/5) = 0.2
    assert abs(oracle.error_rate([0.3, 0.1, 0.2, 0.2, 0.2], [0.2] * 5) - 0.2) < 1e-15


# ------------------------------------------------------------------------------ plan
def compositions(total, parts):
    """All ways to write `total` as an ordered sum of `parts` non-negative integers."""
    if parts == 1:
        yield (total,)
        return
    for first in range(total + 1):
        for rest in compositions(total - first, parts - 1):
            yield (first,) + rest


def check_plan_tables(r, slot_off, slot_expert, S):
    E = len(r)
    assert (r >= 1).all() and slot_off[0] == 0
    assert np.array_equal(np.diff(slot_off), r)
    for e in range(E):
        assert (slot_expert[slot_off[e]:slot_off[e + 1]] == e).all()
    assert (slot_expert[slot_off[E]:] == -1).all()
    assert slot_off[E] <= S


def test_plan_minmax_optimal_brute_force():
    from fractions import Fraction
    for E in (1, 2, 3, 4, 5):
        for extra in range(0, 6):
            for _ in range(6):
                n = rng.integers(0, 40, size=E)
                r, so, se, bound = oracle.plan(n, E + extra)
                check_plan_tables(r, so, se, E + extra)
                assert r.sum() == E + extra
                got = max(Fraction(int(n[e]), int(r[e])) for e in range(E))
                best = min(max(Fraction(int(n[e]), 1 + c[e]) for e in range(E))
                           for c in compositions(extra, E))
                assert got == best
                assert bound == max(-(-int(n[e]) // int(r[e])) for e in range(E))


def test_plan_proportional_closed_form():
    # predicted counts proportional to an integer composition of S: the balanced plan is that
    # composition (Algorithm 1 stops when all devices carry the same load).
    for c in (1, 7, 1000):
        r, so, se, bound = oracle.plan(np.array([9, 1, 1, 1]) * c, 12)
        assert r.tolist() == [9, 1, 1, 1] and bound == c
    m = np.array([3, 1, 4, 1, 5, 2])
    r, _, _, bound = oracle.plan(m * 13, int(m.sum()))
    assert r.tolist() == m.tolist() and bound == 13


def test_plan_hand_worked_ties_and_order():
    assert oracle.plan([4, 2], 3)[0].tolist() == [2, 1]
    assert oracle.plan([2, 2], 3)[0].tolist() == [2, 1]          # equal ratio, equal r: lower index
    assert oracle.plan([4, 2], 4)[0].tolist() == [2, 2]          # 4/2 = 2/1: smaller r wins
    assert oracle.plan([0, 0, 0], 8)[0].tolist() == [3, 3, 2]    # all-zero prediction: round robin
    r, so, se, bound = oracle.plan([5, 0, 1], 5)
    assert r.tolist() == [3, 1, 1] and so.tolist() == [0, 3, 4, 5]
    assert se.tolist() == [0, 0, 0, 1, 2] and bound == 2
    assert oracle.plan([3, 3, 3], 3)[0].tolist() == [1, 1, 1]    # S = E: no duplication


def test_plan_copy_cap():
    r, so, se, bound = oracle.plan([100, 1, 1], 8, c_max=3)
    assert r.tolist() == [3, 3, 2]
    r, so, se, bound = oracle.plan([100, 1], 8, c_max=2)
    assert r.tolist() == [2, 2] and se.tolist() == [0, 0, 1, 1, -1, -1, -1, -1]
    assert bound == 50
    check_plan_tables(r, so, se, 8)


def test_plan_bound_sandwich_and_monotone():
    for _ in range(50):
        E = int(rng.integers(2, 40))
        n = rng.integers(0, 5000, size=E)
        N = int(n.sum())
        prev = None
        for S in range(E, E + 12):
            bound = oracle.plan(n, S)[3]
            assert bound >= -(-N // S)
            assert bound <= int(n.max())
            if S > E:
                assert bound <= max(1, -(-N // (S - E))) or N == 0
            if prev is not None:
                assert bound <= prev
            prev = bound


# ------------------------------------------------------------------------------ pack (Algorithm 1)
def pack_invariants(n, home, cap, c_max, placed, share, load):
    E, G = placed.shape
    assert set(np.unique(placed)) <= {0, 1}
    assert np.array_equal(share.sum(axis=1), n)                     # every token is served exactly once
    assert (share >= 0).all() and ((share > 0) <= (placed == 1)).all()   # only by devices that host its expert
    assert all(placed[e, home[e]] == 1 for e in range(E))           # the original copy is never removed
    assert (placed.sum(axis=0) <= cap).all()                        # memory of every device respected
    if c_max > 0:
        assert (placed.sum(axis=1) <= c_max).all()
    assert np.array_equal(load, share.sum(axis=0))


def test_pack_paper_duplication_example():
    with open(os.path.join(HERE, "golden", "duplication_example.txt")) as f:
        line = [ln for ln in f if not ln.startswith("#")][0]
    tokens, gpus, final = [part.split() for part in line.split("|")]
    n, G = [int(v) for v in tokens], int(gpus[0])
    placed, share, load, iters = oracle.pack(n, list(range(G)), [G] * G)
    assert load.tolist() == [int(final[0])] * G                      # every GPU ends with the same load
    assert placed[0].tolist() == [1] * G and placed[1:].sum() == 3   # only the popular expert is replicated
    pack_invariants(np.array(n), list(range(G)), [G] * G, 0, placed, share, load)


def test_pack_hand_worked_moves():
    # ceil in Delta: loads (5, 0) -> Delta = 3 -> (2, 3); a floor would stop at (3, 2)
    placed, share, load, iters = oracle.pack([5, 0], [0, 1], [2, 2])
    assert load.tolist() == [2, 3] and iters == 1 and share.tolist() == [[2, 3], [0, 0]]
    # ties: two hottest devices (0 and 1) and two coldest (2 and 3): device 0 gives to device 2 first
    placed, share, load, iters = oracle.pack([4, 4, 0, 0], [0, 1, 2, 3], [2, 2, 2, 2])
    assert share.tolist() == [[2, 0, 2, 0], [0, 2, 0, 2], [0, 0, 0, 0], [0, 0, 0, 0]] and iters == 2
    # the biggest expert of the hottest device moves, and the lowest index among equally big ones
    placed, share, load, iters = oracle.pack([3, 3, 1], [0, 0, 0], [3, 3], max_iters=1)
    assert share.tolist() == [[0, 3], [3, 0], [1, 0]]                # Delta = ceil(7/2) = 4, but expert 0 has only 3
    # nothing to do: one device, or loads already within one token
    assert oracle.pack([7, 2], [0, 0], [2])[3] == 0
    assert oracle.pack([3, 4], [0, 1], [2, 2])[3] == 0


def test_pack_reaches_the_termination_target_when_unconstrained():
    # with room everywhere and no copy cap every move is legal, so the loop can only end on its
    # own condition: max L - min L <= 1, i.e. the optimum ceil(N / G)
    for trial in range(40):
        E, G = int(rng.integers(1, 20)), int(rng.integers(1, 9))
        n = rng.integers(0, 200, size=E) * rng.integers(0, 2, size=E)
        home = rng.integers(0, G, size=E)
        placed, share, load, iters = oracle.pack(n, home, [E] * G)
        assert load.max() - load.min() <= 1
        assert load.max() == -(-int(n.sum()) // G)
        pack_invariants(n, home, [E] * G, 0, placed, share, load)


def optimal_max_load(n, home, cap, c_max):
    """Brute force over every placement that keeps the original copies and respects memory and the
    copy cap; for a fixed placement the best achievable max load is found by trying every way of
    splitting every expert's tokens over its hosts (tiny inputs only)."""
    import itertools
    E, G = len(n), len(cap)
    best = None
    options = []
    for e in range(E):
        opts = []
        for mask in range(1 << G):
            if not (mask >> home[e]) & 1:
                continue
            if c_max > 0 and bin(mask).count("1") > c_max:
                continue
            opts.append(mask)
        options.append(opts)
    for masks in itertools.product(*options):
        if any(sum((m >> g) & 1 for m in masks) > cap[g] for g in range(G)):
            continue
        splits = []
        for e in range(E):
            hosts = [g for g in range(G) if (masks[e] >> g) & 1]
            ways = [w for w in itertools.product(range(n[e] + 1), repeat=len(hosts)) if sum(w) == n[e]]
            splits.append([(hosts, w) for w in ways])
        for combo in itertools.product(*splits):
            load = [0] * G
            for hosts, w in combo:
                for g, k in zip(hosts, w):
                    load[g] += k
            m = max(load)
            best = m if best is None or m < best else best
    return best


def test_pack_against_brute_force_on_tiny_inputs():
    cases = 0
    for trial in range(60):
        E, G = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        n = [int(v) for v in rng.integers(0, 5, size=E)]
        home = [int(v) for v in rng.integers(0, G, size=E)]
        homed = [home.count(g) for g in range(G)]
        cap = [homed[g] + int(rng.integers(0, 3)) for g in range(G)]
        c_max = int(rng.integers(0, 3))
        placed, share, load, iters = oracle.pack(n, home, cap, c_max)
        pack_invariants(np.array(n), home, cap, c_max, placed, share, load)
        opt = optimal_max_load(n, home, cap, c_max)
        initial = max(sum(n[e] for e in range(E) if home[e] == g) for g in range(G))
        assert opt <= load.max() <= initial          # a heuristic: never better than the optimum, never worse than doing nothing
        if c_max == 0 and all(c >= E for c in cap):
            assert load.max() == opt                 # unconstrained it is optimal
        cases += 1
    assert cases == 60


def test_pack_respects_copy_cap_and_memory():
    n = [1000, 10, 10, 10]
    # c_max = 1: nothing may be copied, and a token can only go where its expert is: nothing moves
    placed, share, load, iters = oracle.pack(n, [0, 1, 2, 3], [4] * 4, c_max=1)
    assert iters == 0 and share.tolist() == np.diag(n).tolist()
    # c_max = 2: the hot expert gets exactly one more copy
    placed, share, load, iters = oracle.pack(n, [0, 1, 2, 3], [4] * 4, c_max=2)
    assert placed[0].sum() == 2 and load.max() == 505
    # no free place anywhere: same as no copies
    placed, share, load, iters = oracle.pack(n, [0, 1, 2, 3], [1] * 4)
    assert iters == 0 and placed.sum() == 4
    with pytest.raises(ValueError):
        oracle.pack(n, [0, 0, 0, 0], [3, 4, 4, 4])   # initial placement does not fit


def test_pack_never_beats_the_slot_planner_bound():
    # one replica per device (capacity 1, S = G devices, the experts on the first E): this is the
    # setting of plan(), whose greedy is min-max optimal there: Algorithm 1 can match it, not beat it
    for trial in range(20):
        E, extra = int(rng.integers(1, 8)), int(rng.integers(0, 8))
        n = rng.integers(0, 500, size=E)
        G = E + extra
        placed, share, load, iters = oracle.pack(n, list(range(E)), [1] * G)
        _, _, _, bound = oracle.plan(n, G)
        assert load.max() >= bound
        pack_invariants(n, list(range(E)), [1] * G, 0, placed, share, load)
    # one expert, three devices: 100 -> 50/50/0 -> 50/25/25 -> ... the loop keeps shifting tokens
    # between the copies until the loads are within one token
    placed, share, load, iters = oracle.pack([100], [0], [1, 1, 1])
    assert sorted(load.tolist()) == [33, 33, 34] and iters > 2


def test_pack_slots_and_split_by_share():
    # hand-worked: 10 pairs over copies with predicted shares 3 : 1 -> boundaries 0, floor(10*3/4) = 7, 10
    assert oracle.replica_starts_by_share(10, [3, 1]) == [0, 7, 10]
    assert oracle.replica_starts_by_share(10, [0, 5, 0]) == [0, 0, 10, 10]          # a copy with no share gets nothing
    assert oracle.replica_starts_by_share(10, [0, 0, 0]) == oracle.replica_starts(10, 3)   # nothing predicted: even split
    for n in (0, 1, 7, 100, 12345):
        for r in (1, 2, 3, 7):
            assert oracle.replica_starts_by_share(n, [5] * r) == oracle.replica_starts(n, r)  # equal shares = balanced split
    for trial in range(50):
        r, n = int(rng.integers(1, 9)), int(rng.integers(0, 5000))
        sh = rng.integers(0, 1000, size=r)
        st = oracle.replica_starts_by_share(n, sh)
        assert st[0] == 0 and st[-1] == n and all(a <= b for a, b in zip(st, st[1:]))
        if sh.sum() > 0:                                  # every copy within one pair of its proportional part
            loads = np.diff(st)
            assert np.abs(loads - n * sh / sh.sum()).max() < 1.0
    # slot tables of the paper's example: expert 0 on all four devices, the others at home
    placed, share, load, _ = oracle.pack([9, 1, 1, 1], [0, 1, 2, 3], [4] * 4)
    rep, so, se, ss, sd = oracle.pack_slots(placed, share, 9)
    assert rep.tolist() == [4, 1, 1, 1] and so.tolist() == [0, 4, 5, 6, 7]
    assert se.tolist() == [0, 0, 0, 0, 1, 2, 3, -1, -1] and sd.tolist() == [0, 1, 2, 3, 1, 2, 3, -1, -1]
    assert ss.tolist() == [3, 2, 2, 2, 1, 1, 1, 0, 0]
    assert [int(ss[sd == g].sum()) for g in range(4)] == load.tolist()      # shares per device add up to its load
    with pytest.raises(ValueError):
        oracle.pack_slots(placed, share, 6)


def test_dispatch_by_share_realises_the_packed_loads():
    """pack -> pack_slots -> dispatch with shares: with an exact prediction every device receives
    exactly the load Algorithm 1 planned for it, and the permutation keeps all dispatch invariants."""
    E, G, K, T = 6, 3, 2, 300
    idx = random_routing(T, K, E, 1.3)
    n = oracle.histogram(idx, E)
    placed, share, load, _ = oracle.pack(n, [e % G for e in range(E)], [4] * G)
    S = int(placed.sum()) + 2
    rep, so, se, ss, sd = oracle.pack_slots(placed, share, S)
    sro, rp, pr, _ = oracle.dispatch(None, idx, n, rep, so, S, 4, slot_share=ss)
    flat = idx.reshape(-1)
    assert sorted(pr.reshape(-1).tolist()) == sorted(np.nonzero(rp >= 0)[0].tolist())      # bijection onto occupied rows
    assert np.array_equal(rp[pr.reshape(-1)], np.arange(T * K))
    dev_load = np.zeros(G, dtype=np.int64)
    for s in range(S):
        rows = rp[sro[s]:sro[s + 1]]
        rows = rows[rows >= 0]
        assert (np.diff(rows) > 0).all()                                                    # stable inside a slot
        if rows.size:
            assert (flat[rows] == se[s]).all()
            dev_load[sd[s]] += rows.size
        assert rows.size == ss[s]                                                           # exact prediction: planned = realised
    assert dev_load.tolist() == load.tolist() and load.max() - load.min() <= 1
    # with a wrong prediction the split follows the predicted proportions of the ACTUAL counts
    n2 = oracle.histogram(random_routing(T, K, E, 0.2), E)
    idx2 = random_routing(T, K, E, 0.2)
    sro2, rp2, _, _ = oracle.dispatch(None, idx2, oracle.histogram(idx2, E), rep, so, S, 1, slot_share=ss)
    for e in range(E):
        got = [int(np.count_nonzero(rp2[sro2[s]:sro2[s + 1]] >= 0)) for s in range(so[e], so[e + 1])]
        want = np.diff(oracle.replica_starts_by_share(int(oracle.histogram(idx2, E)[e]), ss[so[e]:so[e + 1]])).tolist()
        assert got == want


# ------------------------------------------------------------------------------ dispatch
def closed_form_replica(i, n, r):
    return ((i + 1) * r - 1) // n


def random_routing(T, K, E, skew=1.0):
    p = 1.0 / np.arange(1, E + 1) ** skew
    p /= p.sum()
    idx = np.stack([rng.choice(E, size=K, replace=False, p=p) for _ in range(T)]).astype(np.int32)
    return idx


@pytest.mark.parametrize("T,K,E,S,A", [(50, 2, 4, 4, 1), (50, 2, 4, 9, 1), (97, 3, 7, 12, 8),
                                       (64, 1, 5, 5, 128), (33, 4, 4, 16, 4), (0, 2, 3, 5, 2)])
def test_dispatch_invariants(T, K, E, S, A):
    idx = random_routing(T, K, E, 1.3) if T else np.zeros((0, K), dtype=np.int32)
    hist = oracle.histogram(idx, E)
    r, so, se, bound = oracle.plan(hist, S)            # perfect prediction
    D = 6
    x = rng.integers(0, 1 << 16, size=(T, D), dtype=np.uint16)
    sro, row_pair, pair_row, xp = oracle.dispatch(x, idx, hist, r, so, S, A)
    R = T * K
    Rcap = R + S * (A - 1)
    assert row_pair.shape == (Rcap,) and pair_row.shape == (T, K) and xp.shape == (Rcap, D)
    flat_rows = pair_row.reshape(-1)
    # bijection between pairs and occupied rows
    assert len(set(flat_rows.tolist())) == R
    assert np.array_equal(row_pair[flat_rows], np.arange(R))
    assert (row_pair >= 0).sum() == R
    # slot structure
    assert sro[0] == 0 and (np.diff(sro) >= 0).all() and (sro[:-1] % A == 0).all()
    loads = []
    for s in range(S):
        rows = np.arange(sro[s], sro[s + 1])
        occ = rows[row_pair[rows] >= 0]
        loads.append(len(occ))
        if len(occ):
            assert occ[0] == sro[s] and np.array_equal(occ, np.arange(sro[s], sro[s] + len(occ)))
            pairs = row_pair[occ]
            assert (np.diff(pairs) > 0).all()                       # stable inside a slot
            assert (idx.reshape(-1)[pairs] == se[s]).all()          # right expert
    for e in range(E):
        mine = loads[so[e]:so[e + 1]]
        assert sum(mine) == hist[e]
        assert all(l in (hist[e] // r[e], -(-hist[e] // r[e])) for l in mine)
    assert max(loads + [0]) == (bound if R else 0)                  # perfect prediction: tight
    # replica of a pair follows the closed form floor(((i+1) r - 1) / n)
    seen = [0] * E
    for p in range(R):
        e = int(idx.reshape(-1)[p])
        rho = closed_form_replica(seen[e], int(hist[e]), int(r[e]))
        seen[e] += 1
        assert sro[so[e] + rho] <= flat_rows[p] < sro[so[e] + rho + 1]
    # rows are bit copies
    for p in range(R):
        assert np.array_equal(xp[flat_rows[p]], x[p // K])


def test_dispatch_is_stable_sort_when_unreplicated():
    T, K, E = 200, 2, 8
    idx = random_routing(T, K, E, 1.0)
    hist = oracle.histogram(idx, E)
    r, so, se, _ = oracle.plan(hist, E)
    sro, row_pair, pair_row, _ = oracle.dispatch(None, idx, hist, r, so, E, 1)
    order = np.argsort(idx.reshape(-1), kind="stable")
    assert np.array_equal(row_pair, order)
    assert np.array_equal(sro, np.concatenate([[0], np.cumsum(hist)]))


def test_dispatch_load_bound_under_misprediction():
    # slot load <= ceil((1 + delta_e) * predicted_e / r_e): the slot-level form of the paper's
    # "typical" (1 + eps) * average model of Section 3.3.
    T, K, E, S = 400, 2, 8, 14
    idx = random_routing(T, K, E, 1.2)
    hist = oracle.histogram(idx, E)
    pred = np.maximum(1, np.round(hist * (1 + 0.2 * rng.normal(size=E)))).astype(np.int64)
    r, so, se, bound = oracle.plan(pred, S)
    sro, row_pair, _, _ = oracle.dispatch(None, idx, hist, r, so, S, 1)
    loads = np.diff(sro)
    for e in range(E):
        delta = max(0.0, hist[e] / pred[e] - 1.0)
        for s in range(so[e], so[e + 1]):
            assert loads[s] <= math.ceil((1 + delta) * pred[e] / r[e] + 1e-9)


def test_dispatch_rejects_wrong_hist():
    idx = random_routing(10, 2, 4)
    hist = oracle.histogram(idx, 4)
    hist[0] += 1
    with pytest.raises(ValueError):
        oracle.dispatch(None, idx, hist, [1] * 4, [0, 1, 2, 3, 4], 4, 1)


# ------------------------------------------------------------------------------ expert_ffn / combine
def tiny_layer(T=24, D=16, F=24, E=4, K=2):
    x = to_bf16_bits(rng.normal(size=(T, D)))
    wr = to_bf16_bits(rng.normal(size=(E, D)) / math.sqrt(D))
    b = rng.normal(size=E).astype(np.float32)
    w1 = to_bf16_bits(rng.normal(size=(E, F, D)) * 0.3)
    w3 = to_bf16_bits(rng.normal(size=(E, F, D)) * 0.3)
    w2 = to_bf16_bits(rng.normal(size=(E, D, F)) * 0.3)
    return x, wr, b, w1, w3, w2


def dense_then_mask(x, wr, b, w1, w3, w2, K, mode):
    """Every expert on every token with torch's own SiLU, then the K-sparse gate matrix."""
    X = torch.from_numpy(oracle.bf16_bits_to_f64(x))
    E = wr.shape[0]
    idx, w, _ = oracle.route(x, wr, b, K, mode)
    gate = torch.zeros(X.shape[0], E, dtype=torch.float64)
    for t in range(X.shape[0]):
        for j in range(K):
            gate[t, idx[t, j]] = w[t, j]
    out = torch.zeros(X.shape[0], w2.shape[1], dtype=torch.float64)
    for e in range(E):
        W1 = torch.from_numpy(oracle.bf16_bits_to_f64(w1[e]))
        W3 = torch.from_numpy(oracle.bf16_bits_to_f64(w3[e]))
        W2 = torch.from_numpy(oracle.bf16_bits_to_f64(w2[e]))
        y = (torch.nn.functional.silu(X @ W1.T) * (X @ W3.T)) @ W2.T
        out += gate[:, e:e + 1] * y
    return out.numpy()


@pytest.mark.parametrize("S,A,mode,pred", [(4, 1, 0, "true"), (7, 1, 0, "zero"), (9, 4, 1, "true"),
                                           (6, 128, 0, "skewed")])
def test_layer_equals_dense_all_experts_then_mask(S, A, mode, pred):
    x, wr, b, w1, w3, w2 = tiny_layer()
    E, K = 4, 2
    true_hist = oracle.histogram(oracle.route(x, wr, b, K, mode)[0], E)
    pred_hist = {"true": true_hist, "zero": np.zeros(E, dtype=np.int64),
                 "skewed": np.array([100, 0, 3, 1])}[pred]
    res = oracle.moe_layer(x, wr, b, w1, w3, w2, pred_hist, K=K, S=S, gate_mode=mode, row_align=A)
    want = dense_then_mask(x, wr, b, w1, w3, w2, K, mode)
    assert np.allclose(res["out"], want, rtol=1e-10, atol=1e-12)
    assert res["hist"].sum() == x.shape[0] * K


def test_layer_output_independent_of_placement():
    x, wr, b, w1, w3, w2 = tiny_layer()
    base = oracle.moe_layer(x, wr, b, w1, w3, w2, [1, 1, 1, 1], K=2, S=4)["out"]
    for S, A, c_max, pred in [(11, 1, 0, [50, 1, 1, 1]), (8, 16, 2, [0, 9, 0, 9]), (5, 3, 0, [1, 2, 3, 4])]:
        out = oracle.moe_layer(x, wr, b, w1, w3, w2, pred, K=2, S=S, row_align=A, c_max=c_max)["out"]
        assert np.allclose(out, base, rtol=1e-12, atol=1e-14)


def test_ffn_single_expert_is_a_dense_mlp():
    T, D, F = 10, 8, 12
    xp = to_bf16_bits(rng.normal(size=(T, D)))
    w1 = to_bf16_bits(rng.normal(size=(1, F, D)))
    w3 = to_bf16_bits(rng.normal(size=(1, F, D)))
    w2 = to_bf16_bits(rng.normal(size=(1, D, F)))
    yp = oracle.expert_ffn(xp, [0, T], [0], w1, w3, w2)
    X = torch.from_numpy(oracle.bf16_bits_to_f64(xp))
    lin1 = torch.nn.Linear(D, F, bias=False, dtype=torch.float64)
    lin3 = torch.nn.Linear(D, F, bias=False, dtype=torch.float64)
    lin2 = torch.nn.Linear(F, D, bias=False, dtype=torch.float64)
    with torch.no_grad():
        lin1.weight.copy_(torch.from_numpy(oracle.bf16_bits_to_f64(w1[0])))
        lin3.weight.copy_(torch.from_numpy(oracle.bf16_bits_to_f64(w3[0])))
        lin2.weight.copy_(torch.from_numpy(oracle.bf16_bits_to_f64(w2[0])))
        want = lin2(torch.nn.functional.silu(lin1(X)) * lin3(X)).numpy()
    assert np.allclose(yp, want, rtol=1e-12, atol=1e-14)


def test_ffn_zero_weights_and_row_subset():
    T, D, F, E = 12, 8, 10, 3
    xp = to_bf16_bits(rng.normal(size=(T, D)))
    w1 = to_bf16_bits(rng.normal(size=(E, F, D)))
    w3 = to_bf16_bits(rng.normal(size=(E, F, D)))
    w2 = to_bf16_bits(rng.normal(size=(E, D, F)))
    off, se = [0, 5, 5, 12], [2, 0, 1]
    full = oracle.expert_ffn(xp, off, se, w1, w3, w2)
    assert np.abs(full).max() > 0
    assert not oracle.expert_ffn(xp, off, se, np.zeros_like(w1), w3, w2).any()   # silu(0) = 0
    assert not oracle.expert_ffn(xp, off, se, w1, w3, np.zeros_like(w2)).any()
    part = oracle.expert_ffn(xp, off, se, w1, w3, w2, rows=[1, 7, 11])
    assert np.allclose(part[[1, 7, 11]], full[[1, 7, 11]], rtol=1e-12, atol=0)
    assert not part[[0, 2, 3, 4, 5, 6, 8, 9, 10]].any()
    # each slot uses its own expert: swapping the experts of two slots changes those rows only
    swapped = oracle.expert_ffn(xp, off, [1, 0, 2], w1, w3, w2)
    assert not np.allclose(swapped, full)


def test_combine_identity_gather_and_linearity():
    T, K, E, D = 40, 3, 6, 8
    idx = random_routing(T, K, E)
    hist = oracle.histogram(idx, E)
    r, so, se, _ = oracle.plan(hist, 9)
    x = to_bf16_bits(rng.normal(size=(T, D)))
    sro, row_pair, pair_row, xp = oracle.dispatch(x, idx, hist, r, so, 9, 4)
    w = rng.random(size=(T, K))
    w /= w.sum(axis=1, keepdims=True)
    # Yp := Xp with weights that sum to one gives back X
    out = oracle.combine(xp, pair_row, w)
    assert np.allclose(out, oracle.bf16_bits_to_f64(x), rtol=1e-12, atol=1e-15)
    # K = 1: a pure gather
    out1 = oracle.combine(xp, pair_row[:, :1], np.ones((T, 1)))
    assert np.array_equal(out1, oracle.bf16_bits_to_f64(x))
    # linear in the weights, and a hand-checkable case
    yp = rng.normal(size=(xp.shape[0], D))
    w2 = rng.random(size=(T, K))
    assert np.allclose(oracle.combine(yp, pair_row, 2 * w + 3 * w2),
                       2 * oracle.combine(yp, pair_row, w) + 3 * oracle.combine(yp, pair_row, w2))
    small = oracle.combine(np.array([[1.0, 10.0], [2.0, 20.0], [4.0, 40.0]]),
                           np.array([[2, 0]]), np.array([[0.25, 0.5]]))
    assert small.tolist() == [[1.5, 15.0]]
    sub = oracle.combine(yp, pair_row, w, tokens=[3, 17])
    assert np.array_equal(sub[[3, 17]], oracle.combine(yp, pair_row, w)[[3, 17]])


# ------------------------------------------------------------------------------ predictor state
def test_predictor_state_is_the_pooled_mle_and_a_moving_average():
    E, K = 7, 2
    batches = [random_routing(T, K, E, 1.1) for T in (40, 40, 40, 40)]
    state = [0] * E
    for b in batches:
        state, pred = oracle.predictor_update(state, oracle.histogram(b, E))
    pooled = np.bincount(np.concatenate([b.reshape(-1) for b in batches]), minlength=E)
    assert state == pooled.tolist() and pred.tolist() == pooled.tolist()
    # Eq. 1 over the pooled tokens; with equal batch sizes that is the plain average of the per-batch estimates
    per_batch = np.mean([oracle.p_hat(oracle.histogram(b, E)) for b in batches], axis=0)
    assert np.allclose(oracle.p_hat(pred), per_batch, rtol=1e-12)
    assert abs(oracle.p_hat(pred).sum() - 1) < 1e-12


def test_predictor_scales_huge_counts_by_a_power_of_two():
    state, pred = oracle.predictor_update([2 ** 33, 2 ** 31, 3], [0, 0, 1])
    assert state == [2 ** 33, 2 ** 31, 4]
    assert pred.tolist() == [2 ** 30, 2 ** 28, 0]          # shifted right by 3: the largest fits 31 bits
    state, pred = oracle.predictor_update([2 ** 31 - 2, 5], [1, 0])
    assert pred.tolist() == [2 ** 31 - 1, 5]               # still fits: no scaling
    with pytest.raises(ValueError):
        oracle.predictor_update([1, 1], [0, -1])


def test_predictor_ema_special_cases_and_closed_form():
    from fractions import Fraction
    # alpha = 1 (shift 0): the state is the last batch, in units of 2^-16 tokens
    state, pred = oracle.predictor_update_ema([123456, 7], [10, 20], 0)
    assert state == [10 << 16, 20 << 16]
    # a constant input is a fixed point, whatever the weight
    for shift in (1, 3, 8, 16):
        state, _ = oracle.predictor_update_ema([5 << 16, 0, 777 << 16], [5, 0, 777], shift)
        assert state == [5 << 16, 0, 777 << 16]
    # against the exact recurrence s_t = s_{t-1} + (h_t 2^16 - s_{t-1}) / 2^k in rationals: every step
    # floors once, and the error it leaves decays like the state does, so the two stay within 2^k units
    seq = rng.integers(0, 100000, size=(40, 6))
    for shift in (1, 2, 5):
        state, exact = [0] * 6, [Fraction(0)] * 6
        for h in seq:
            state, pred = oracle.predictor_update_ema(state, h, shift)
            exact = [x + (Fraction(int(v) << 16) - x) / 2 ** shift for x, v in zip(exact, h)]
            assert all(0 <= float(x - s) <= 2 ** shift for x, s in zip(exact, state))
        # the textbook form: a geometrically weighted sum of the inputs
        a = Fraction(1, 2 ** shift)
        closed = [sum(a * (1 - a) ** (len(seq) - 1 - i) * (int(seq[i][e]) << 16) for i in range(len(seq))) for e in range(6)]
        assert all(abs(float(c - x)) < 1e-6 for c, x in zip(closed, exact))
    # proportions: two experts fed in the ratio 3:1 are predicted in that ratio
    state = [0, 0]
    for _ in range(200):
        state, pred = oracle.predictor_update_ema(state, [3000, 1000], 4)
    assert abs(pred[0] / pred[1] - 3.0) < 1e-3
    # a step in the input is followed monotonically, and old batches are forgotten (unlike the cumulative form)
    state, seen = [1000 << 16], []
    for _ in range(60):
        state, pred = oracle.predictor_update_ema(state, [0], 2)
        seen.append(state[0])
    assert seen == sorted(seen, reverse=True) and seen[-1] < (1 << 16) // 100
    with pytest.raises(ValueError):
        oracle.predictor_update_ema([0], [1], 17)
