"""Plain CPU statement of the six steps of the MoE hot path, in numpy / fp64.

TEST INFRASTRUCTURE ONLY: never imported by the product package.  Nothing here is blocked, fused,
vectorised for speed or tuned; every function is the definition of its step written out so that it
can be checked against the paper by eye.  Library primitives used as steps: an fp64 matmul and a
stable sort.

Parity status: every function below is pinned by tests that do not restate its formula (closed
forms, brute force on tiny inputs, textbook special cases, the paper's worked skewness example);
none is "parity unpinned".

Notation (paper, Section 2 and Algorithm 1): T tokens, D model width, F expert hidden width,
E experts, K experts per token, S logical slots (the "GPUs" of Algorithm 1, one expert replica
each), R = T*K routed (token, choice) pairs with flat index p = t*K + j, A = row alignment of a
slot's first row.

bf16 tensors are passed as numpy uint16 bit patterns (the upper half of an IEEE fp32); arrays of
any float dtype are taken as already-decoded values.  All floating-point work is done in fp64.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "bf16_bits_to_f64", "route_logits", "route", "histogram", "p_hat", "skewness", "error_rate",
    "predictor_update", "predictor_update_ema",
    "plan", "pack", "pack_slots", "replica_starts", "replica_starts_by_share", "dispatch", "expert_ffn",
    "combine", "moe_layer",
]


# --------------------------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Decode bfloat16 bit patterns (uint16) to fp64.  bf16 is the top 16 bits of an fp32, so the
    conversion is exact."""
    bits = np.ascontiguousarray(bits)
    if bits.dtype != np.uint16:
        raise TypeError("bf16 bit patterns must be uint16")
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _values(a: np.ndarray) -> np.ndarray:
    """fp64 values of `a`: uint16 is read as bf16 bits, floats are widened."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return bf16_bits_to_f64(a)
    if a.dtype.kind != "f":
        raise TypeError(f"expected bf16 bits (uint16) or a float array, got {a.dtype}")
    return a.astype(np.float64)


# --------------------------------------------------------------------------------------------
# route  (Section 2: every token is sent to its top-K experts; the mapping is never altered)
# --------------------------------------------------------------------------------------------
def route_logits(x, w_router, bias=None) -> np.ndarray:
    """logit[t, e] = sum_d X[t, d] * Wr[e, d] + b[e]   (fp64)."""
    X = _values(x)
    Wr = _values(w_router)
    if X.ndim != 2 or Wr.ndim != 2 or X.shape[1] != Wr.shape[1]:
        raise ValueError("x is [T, D], w_router is [E, D]")
    logits = X @ Wr.T
    if bias is not None:
        b = np.asarray(bias, dtype=np.float64)
        if b.shape != (Wr.shape[0],):
            raise ValueError("bias is [E]")
        logits = logits + b[None, :]
    return logits


def route(x, w_router, bias, K: int, gate_mode: int = 0):
    """Top-K routing of Section 2.

    Selection: the K largest logits of each token, listed in descending logit order; equal logits
    are ordered by ascending expert index.  The choice is always made on the logits (the sigmoid of
    mode 1 is monotone, so it selects the same experts).

    Gate weights over the selected experts only:
      gate_mode 0: softmax,  w_j = exp(l_j - l_max) / sum_i exp(l_i - l_max)
      gate_mode 1: sigmoid then renormalise,  s_j = 1 / (1 + exp(-l_j)),  w_j = s_j / sum_i s_i

    Returns (topk_idx int32 [T, K], topk_w fp64 [T, K], logits fp64 [T, E]).
    """
    logits = route_logits(x, w_router, bias)
    T, E = logits.shape
    if not (1 <= K <= E):
        raise ValueError("need 1 <= K <= E")
    if gate_mode not in (0, 1):
        raise ValueError("gate_mode is 0 (softmax) or 1 (sigmoid)")
    # A stable ascending sort of the negated logits lists experts by descending logit and keeps
    # equal logits in ascending expert order.
    order = np.argsort(-logits, axis=1, kind="stable")
    topk_idx = order[:, :K].astype(np.int32)
    sel = np.take_along_axis(logits, topk_idx.astype(np.int64), axis=1)
    if gate_mode == 0:
        z = np.exp(sel - sel[:, :1])          # sel[:, 0] is the row maximum
        topk_w = z / z.sum(axis=1, keepdims=True)
    else:
        s = 1.0 / (1.0 + np.exp(-sel))
        topk_w = s / s.sum(axis=1, keepdims=True)
    return topk_idx, topk_w, logits


# --------------------------------------------------------------------------------------------
# histogram and the load statistics built on it  (Eq. 1; "Quantifying Imbalance"; error rate)
# --------------------------------------------------------------------------------------------
def histogram(topk_idx, E: int) -> np.ndarray:
    """n_e = number of routed pairs whose expert is e (the n_i of Eq. 1 with N = T*K)."""
    idx = np.asarray(topk_idx).reshape(-1)
    if idx.size and (idx.min() < 0 or idx.max() >= E):
        raise ValueError("expert index out of range")
    return np.array([int(np.count_nonzero(idx == e)) for e in range(E)], dtype=np.int64)


def p_hat(hist) -> np.ndarray:
    """Eq. 1: the maximum-likelihood estimate p_i = n_i / N."""
    h = np.asarray(hist, dtype=np.float64)
    return h / h.sum()


def skewness(hist) -> float:
    """Load of the most popular expert divided by the load every expert would have if the tokens
    were spread evenly (Section 2, "Quantifying Imbalance")."""
    h = np.asarray(hist, dtype=np.float64)
    return float(h.max() / (h.sum() / h.size))


def error_rate(p_est, p_true) -> float:
    """|p_est - p_true| measured in units of 1/E (Section 3.2.1), averaged over the experts as
    Section 3.3 reads it."""
    a = np.asarray(p_est, dtype=np.float64)
    b = np.asarray(p_true, dtype=np.float64)
    E = a.size
    return float(np.mean(np.abs(a - b) / (1.0 / E)))


def predictor_update(state, hist):
    """Distribution-Only predictor state over batches (Section 3.2.1, the estimate of Eq. 1
    averaged over the batches seen): the state holds the per-expert counts of all
    batches seen, so state / sum(state) is the maximum-likelihood estimate over the pooled tokens.
    Returns (new_state as Python ints, predicted_hist int32): the prediction handed to the planner
    is the state itself, divided by the smallest power of two that makes its largest entry fit an
    int32 (only proportions matter to the plan)."""
    s = [int(a) + int(b) for a, b in zip(np.asarray(state).reshape(-1), np.asarray(hist).reshape(-1))]
    if any(int(b) < 0 for b in np.asarray(hist).reshape(-1)):
        raise ValueError("counts must be >= 0")
    shift = 0
    while (max(s) >> shift) > 2 ** 31 - 1:
        shift += 1
    return s, np.array([v >> shift for v in s], dtype=np.int32)


def predictor_update_ema(state, hist, shift: int):
    """Exponentially weighted form of the same estimate (Section 3.2.1 speaks of a moving average
    over batches without fixing its weights; the cumulative form above weights all batches alike,
    this one forgets old batches geometrically with alpha = 2^-shift).  Integer arithmetic only:
    the state holds per-expert counts in units of 2^-16 tokens and moves towards the new batch by
    state += floor((hist * 2^16 - state) / 2^shift).  The prediction handed to the planner is the
    state divided by the smallest power of two that makes its largest entry fit an int32 (only
    proportions matter to the plan).  Returns (new_state as Python ints, predicted_hist int32)."""
    if not (0 <= int(shift) <= 16):
        raise ValueError("shift in 0..16")
    h = [int(b) for b in np.asarray(hist).reshape(-1)]
    if any(b < 0 for b in h):
        raise ValueError("counts must be >= 0")
    s = [int(a) + (((b << 16) - int(a)) >> int(shift)) for a, b in zip(np.asarray(state).reshape(-1), h)]
    down = 0
    while (max(s) >> down) > 2 ** 31 - 1:
        down += 1
    return s, np.array([v >> down for v in s], dtype=np.int32)


# --------------------------------------------------------------------------------------------
# plan  (Algorithm 1 driven by predicted counts, one expert replica per logical slot)
# --------------------------------------------------------------------------------------------
def plan(pred_hist, S: int, c_max: int = 0):
    """Replica counts from a predicted histogram.

    Algorithm 1 with G = S devices that each hold one expert replica, started from "expert e alone
    on its own slot, S - E slots free": its hottest device is always the replica group with the
    largest per-replica load and its coldest device is a free slot, so each round hands the next
    free slot to the expert with the largest predicted load per replica.  Only proportions are
    predicted (Section 3.2.1), so the plan fixes replica counts; tokens are split later by dispatch.

      r_e = 1 for all e;  S - E times: e* = argmax_e  n_e / r_e  over experts with r_e < c_max
      (c_max = 0: no cap);  r_{e*} += 1.
    Comparison is exact (integers, cross-multiplied); equal ratios go to the smaller r, then to
    the lower expert index.  When no expert is eligible the remaining slots stay empty (-1).

    Returns (replicas [E], slot_off [E+1], slot_expert [S], bound) with expert e owning slots
    slot_off[e] .. slot_off[e+1]-1 and bound = max_e ceil(n_e / r_e).
    """
    n = [int(v) for v in np.asarray(pred_hist).reshape(-1)]
    E = len(n)
    if any(v < 0 for v in n):
        raise ValueError("predicted counts must be >= 0")
    if S < E:
        raise ValueError("need S >= E")
    r = [1] * E
    for _ in range(S - E):
        best = -1
        for e in range(E):
            if c_max > 0 and r[e] >= c_max:
                continue
            if best < 0:
                best = e
                continue
            lhs = n[e] * r[best]          # n_e / r_e  vs  n_best / r_best
            rhs = n[best] * r[e]
            if lhs > rhs or (lhs == rhs and r[e] < r[best]):
                best = e                  # equal ratio and equal r keeps the lower index
        if best < 0:
            break
        r[best] += 1
    slot_off = [0] * (E + 1)
    for e in range(E):
        slot_off[e + 1] = slot_off[e] + r[e]
    slot_expert = [-1] * S
    for e in range(E):
        for s in range(slot_off[e], slot_off[e + 1]):
            slot_expert[s] = e
    bound = max(-(-n[e] // r[e]) for e in range(E))
    return (np.array(r, dtype=np.int32), np.array(slot_off, dtype=np.int32),
            np.array(slot_expert, dtype=np.int32), int(bound))


# --------------------------------------------------------------------------------------------
# pack  (Algorithm 1 itself: G devices with limited memory, several experts per device)
# --------------------------------------------------------------------------------------------
def pack(pred_hist, home, capacity, c_max: int = 0, max_iters: int = 1 << 20):
    """Algorithm 1 on predicted per-expert token counts, in count form.

    Devices g = 0..G-1 can hold capacity[g] expert copies each (all experts have the same number of
    parameters, so the algorithm's memory test "params(e) <= M_g" is a count of free places).  The
    initial placement puts expert e on device home[e] alone, and all its n_e tokens are dispatched
    there (the algorithm's first step: every token goes to the lowest device that hosts its expert).
    Only counts are known before routing (Section 3.2.1), so the dispatch d is kept as
    share[e][g] = number of expert e's tokens served by device g, and "the first Delta tokens" are
    any Delta of them.

    Loop, exactly as printed, while max_g L_g - min_g L_g > 1:
      g_h = argmax L, g_c = argmin L (ties: lowest device);  Delta = ceil((L_gh - L_gc) / 2);
      e* = the expert with the most tokens on g_h (ties: lowest expert) AMONG those that g_c already
           hosts or may receive: copies(e) < c_max (c_max = 0: no cap) and g_c has a free place;
      copy e* to g_c if it is not there;  move min(Delta, share[e*][g_h]) tokens of e* from g_h to g_c.
    The restriction of e* to experts that g_c can serve is the reading taken where the printed
    algorithm is incomplete: as printed, a refused copy would still send tokens to a device without
    the expert.  When no expert of g_h can be served by g_c the loop ends (no legal move for the
    hottest/coldest pair).  Every pass moves between 1 and Delta < L_gh - L_gc tokens, so
    sum_g L_g^2 falls strictly and the loop terminates.

    Returns (placement int32 [E, G] of 0/1, share int64 [E, G], load int64 [G], iterations).
    """
    n = [int(v) for v in np.asarray(pred_hist).reshape(-1)]
    hm = [int(v) for v in np.asarray(home).reshape(-1)]
    cap = [int(v) for v in np.asarray(capacity).reshape(-1)]
    E, G = len(n), len(cap)
    if len(hm) != E or any(v < 0 for v in n) or any(not (0 <= g < G) for g in hm):
        raise ValueError("need counts >= 0 and a home device in [0, G) per expert")
    placed = [[0] * G for _ in range(E)]
    share = [[0] * G for _ in range(E)]
    used = [0] * G
    copies = [1] * E
    for e in range(E):
        placed[e][hm[e]] = 1
        share[e][hm[e]] = n[e]
        used[hm[e]] += 1
    if any(used[g] > cap[g] for g in range(G)):
        raise ValueError("the initial placement exceeds a device's capacity")
    load = [sum(share[e][g] for e in range(E)) for g in range(G)]
    iters = 0
    while iters < max_iters:
        g_h = max(range(G), key=lambda g: (load[g], -g))
        g_c = min(range(G), key=lambda g: (load[g], g))
        if load[g_h] - load[g_c] <= 1:
            break
        delta = -(-(load[g_h] - load[g_c]) // 2)
        best = -1
        for e in range(E):
            if share[e][g_h] <= 0:
                continue
            servable = placed[e][g_c] or ((c_max <= 0 or copies[e] < c_max) and used[g_c] < cap[g_c])
            if servable and (best < 0 or share[e][g_h] > share[best][g_h]):
                best = e
        if best < 0:
            break
        if not placed[best][g_c]:
            placed[best][g_c] = 1
            copies[best] += 1
            used[g_c] += 1
        m = min(delta, share[best][g_h])
        share[best][g_h] -= m
        share[best][g_c] += m
        load[g_h] -= m
        load[g_c] += m
        iters += 1
    return (np.array(placed, dtype=np.int32), np.array(share, dtype=np.int64),
            np.array(load, dtype=np.int64), iters)


def pack_slots(placement, share, S: int):
    """The placement of Algorithm 1 as slot tables: one slot per (expert, device) copy, experts in
    ascending order and, within an expert, its devices in ascending order (the numbering dispatch
    expects: expert e owns slots slot_off[e] .. slot_off[e+1]-1).  slot_share[s] is the number of
    predicted tokens the algorithm's dispatch d assigned to that copy, slot_device[s] its device;
    slots beyond the last copy are empty (expert -1, device -1, share 0).
    Returns (replicas [E], slot_off [E+1], slot_expert [S], slot_share [S], slot_device [S])."""
    P = np.asarray(placement)
    sh = np.asarray(share)
    E, G = P.shape
    replicas = [int(P[e].sum()) for e in range(E)]
    if sum(replicas) > S:
        raise ValueError("more copies than slots")
    slot_off = [0] * (E + 1)
    slot_expert, slot_share, slot_device = [-1] * S, [0] * S, [-1] * S
    for e in range(E):
        slot_off[e + 1] = slot_off[e] + replicas[e]
        s = slot_off[e]
        for g in range(G):
            if P[e][g]:
                slot_expert[s], slot_share[s], slot_device[s] = e, int(sh[e][g]), g
                s += 1
    as_i32 = lambda v: np.array(v, dtype=np.int32)  # noqa: E731
    return as_i32(replicas), as_i32(slot_off), as_i32(slot_expert), as_i32(slot_share), as_i32(slot_device)


# --------------------------------------------------------------------------------------------
# dispatch  (the routing all-to-all of Section 2 on one device; replica choice of Algorithm 1)
# --------------------------------------------------------------------------------------------
def replica_starts(n_e: int, r_e: int):
    """Contiguous balanced split of an expert's n_e pairs over its r_e replicas: replica rho takes
    the stable ranks start[rho] .. start[rho+1]-1 with start[rho] = floor(rho * n_e / r_e)."""
    return [(rho * n_e) // r_e for rho in range(r_e + 1)]


def replica_starts_by_share(n_e: int, shares):
    """Split of an expert's n_e ACTUAL pairs over its copies in proportion to the predicted tokens
    that Algorithm 1's dispatch gave each copy: copy rho takes the stable ranks
    start[rho] .. start[rho+1]-1 with start[rho] = floor(n_e * (shares[0] + .. + shares[rho-1]) / sum).
    Every copy's load is within one pair of its proportional part.  When the prediction gave the
    expert no tokens at all (sum = 0) nothing is known and the split is the balanced one."""
    sh = [int(v) for v in shares]
    tot = sum(sh)
    if tot <= 0:
        return replica_starts(n_e, len(sh))
    cum, out = 0, [0]
    for v in sh:
        cum += v
        out.append((n_e * cum) // tot)
    return out


def dispatch(x, topk_idx, hist, replicas, slot_off, S: int, row_align: int = 1, slot_share=None):
    """Lossless, stable permutation of routed pairs into slot buckets.

    For pair p (expert e = topk_idx[p]) the stable rank is i_p = #{q < p : topk_idx[q] = e}
    ("the first tokens" of Algorithm 1 are taken in flat pair order).  The pair goes to the replica
    rho whose rank range contains i_p, i.e. slot s = slot_off[e] + rho, at row
    slot_row_off[s] + (i_p - start[rho]).  Slot s begins at a multiple of `row_align`;
    slot_row_off[s+1] = round_up(slot_row_off[s] + load_s, row_align).

    With `slot_share` (int [S], from pack_slots) the copies of an expert take shares of its pairs in
    proportion to those predicted counts instead of equal shares (replica_starts_by_share).

    Returns (slot_row_off int32 [S+1], row_pair int32 [Rcap] with -1 on padding rows,
             pair_row int32 [R], Xp [Rcap, D] bit copies of the token rows (zeros on padding)),
    Rcap = R + S*(row_align-1).  x may be None (then Xp is None).
    """
    idx = np.asarray(topk_idx)
    if idx.ndim != 2:
        raise ValueError("topk_idx is [T, K]")
    T, K = idx.shape
    R = T * K
    flat = idx.reshape(-1)
    n = [int(v) for v in np.asarray(hist).reshape(-1)]
    r = [int(v) for v in np.asarray(replicas).reshape(-1)]
    so = [int(v) for v in np.asarray(slot_off).reshape(-1)]
    E = len(n)
    A = int(row_align)
    if A < 1:
        raise ValueError("row_align >= 1")
    if [int(v) for v in histogram(flat, E)] != n:
        raise ValueError("hist does not match topk_idx")

    # load of every slot
    load = [0] * S
    starts = []
    for e in range(E):
        if slot_share is None:
            st = replica_starts(n[e], r[e])
        else:
            st = replica_starts_by_share(n[e], np.asarray(slot_share).reshape(-1)[so[e]:so[e] + r[e]])
        starts.append(st)
        for rho in range(r[e]):
            load[so[e] + rho] = st[rho + 1] - st[rho]
    slot_row_off = [0] * (S + 1)
    for s in range(S):
        end = slot_row_off[s] + load[s]
        slot_row_off[s + 1] = ((end + A - 1) // A) * A
    Rcap = R + S * (A - 1)

    pair_row = np.full(R, -1, dtype=np.int32)
    row_pair = np.full(Rcap, -1, dtype=np.int32)
    seen = [0] * E                               # pairs of expert e met so far = stable rank
    for p in range(R):
        e = int(flat[p])
        i = seen[e]
        seen[e] += 1
        st = starts[e]
        rho = 0
        while not (st[rho] <= i < st[rho + 1]):  # the replica whose rank range holds i
            rho += 1
        row = slot_row_off[so[e] + rho] + (i - st[rho])
        pair_row[p] = row
        row_pair[row] = p

    xp = None
    if x is not None:
        x = np.asarray(x)
        xp = np.zeros((Rcap, x.shape[1]), dtype=x.dtype)
        for p in range(R):
            xp[pair_row[p]] = x[p // K]
    return (np.array(slot_row_off, dtype=np.int32), row_pair, pair_row.reshape(T, K), xp)


# --------------------------------------------------------------------------------------------
# expert_ffn  (expert-parallel SwiGLU FFN of Sections 2 and 3.4, one expert replica per slot)
# --------------------------------------------------------------------------------------------
def expert_ffn(xp, slot_row_off, slot_expert, w_gate, w_up, w_down, rows=None) -> np.ndarray:
    """For every row rho of slot s (expert e = slot_expert[s]):
         g = W1[e] xp[rho],  u = W3[e] xp[rho],  h = silu(g) * u,  Yp[rho] = W2[e] h,
       silu(z) = z / (1 + exp(-z));  no bias terms;  nothing is rounded.
    W1, W3 are [E, F, D] and W2 is [E, D, F] (output features x input features); they are only
    ever indexed by expert, so any container with w[e] -> 2-D array will do.
    All rows of a slot's extent [slot_row_off[s], slot_row_off[s+1]) are computed; `rows`
    restricts the work to the listed rows (others stay 0).  Returns Yp fp64 [Rcap, D]."""
    off = [int(v) for v in np.asarray(slot_row_off).reshape(-1)]
    se = [int(v) for v in np.asarray(slot_expert).reshape(-1)]
    S = len(se)
    xp = np.asarray(xp)
    Rcap = xp.shape[0]
    yp = np.zeros((Rcap, xp.shape[1]), dtype=np.float64)      # the FFN maps D back to D
    want = None if rows is None else np.unique(np.asarray(rows, dtype=np.int64))
    for s in range(S):
        e = se[s]
        lo, hi = off[s], off[s + 1]
        if e < 0 or hi <= lo:
            continue
        sel = np.arange(lo, hi) if want is None else want[(want >= lo) & (want < hi)]
        if sel.size == 0:
            continue
        xs = _values(xp[sel])
        g = xs @ _values(w_gate[e]).T
        u = xs @ _values(w_up[e]).T
        with np.errstate(over="ignore"):
            h = g / (1.0 + np.exp(-g)) * u
        yp[sel] = h @ _values(w_down[e]).T
    return yp


# --------------------------------------------------------------------------------------------
# combine  (the post-FFN shuffle of Section 2: expert outputs return to token order)
# --------------------------------------------------------------------------------------------
def combine(yp, pair_row, topk_w, tokens=None) -> np.ndarray:
    """out[t, :] = sum_{j<K} topk_w[t, j] * Yp[pair_row[t, j], :], summed in ascending j.
    `tokens` restricts the work to the listed tokens (others stay 0).  Returns fp64 [T, D]."""
    pr = np.asarray(pair_row)
    w = np.asarray(topk_w, dtype=np.float64)
    T, K = pr.shape
    yp = np.asarray(yp)
    out = np.zeros((T, yp.shape[1]), dtype=np.float64)
    which = range(T) if tokens is None else [int(t) for t in tokens]
    for t in which:
        acc = np.zeros(yp.shape[1], dtype=np.float64)
        for j in range(K):
            acc = acc + w[t, j] * _values(yp[int(pr[t, j])])
        out[t] = acc
    return out


# --------------------------------------------------------------------------------------------
# the whole layer
# --------------------------------------------------------------------------------------------
def moe_layer(x, w_router, bias, w_gate, w_up, w_down, pred_hist, *, K: int, S: int,
              gate_mode: int = 0, row_align: int = 1, c_max: int = 0) -> dict:
    """plan (from the predicted histogram) -> route -> histogram -> dispatch -> expert_ffn ->
    combine, every intermediate kept in fp64."""
    E = np.asarray(w_router).shape[0]
    replicas, slot_off, slot_expert, bound = plan(pred_hist, S, c_max)
    topk_idx, topk_w, logits = route(x, w_router, bias, K, gate_mode)
    hist = histogram(topk_idx, E)
    slot_row_off, row_pair, pair_row, xp = dispatch(x, topk_idx, hist, replicas, slot_off, S,
                                                    row_align)
    yp = expert_ffn(xp, slot_row_off, slot_expert, w_gate, w_up, w_down)
    out = combine(yp, pair_row, topk_w)
    return dict(replicas=replicas, slot_off=slot_off, slot_expert=slot_expert, bound=bound,
                topk_idx=topk_idx, topk_w=topk_w, logits=logits, hist=hist,
                slot_row_off=slot_row_off, row_pair=row_pair, pair_row=pair_row, xp=xp, yp=yp,
                out=out)
