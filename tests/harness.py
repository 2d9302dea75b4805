"""Shared helpers of the test-suite: seeded inputs with a routing margin, bf16 views, comparisons.

The margin screening lives here (not in the input generators) because it needs the oracle's fp64
logits: a token whose K-th and (K+1)-th (or any two selected) logits are closer than TAU cannot
have a well-defined "exact" top-K under fp32 accumulation, so such rows are re-drawn from a seeded
stream before the inputs are handed to either side.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2506_07366_b200 import workloads as wl

TAU = 2.0 ** -12          # minimum gap between the logits that decide a token's top-K
FLOAT_RTOL_OF_MAX = 2e-2  # float outputs: max|gpu - ref| <= 2e-2 * max|ref|


def bits(t: torch.Tensor) -> np.ndarray:
    return wl.bf16_bits(t)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16).copy()).view(torch.bfloat16).to(device)


def f64_to_bf16_tensor(a: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).to(device)


def token_margins(logits: np.ndarray, K: int) -> np.ndarray:
    """min over the K deciding gaps of each token's descending logits."""
    srt = -np.sort(-logits, axis=1)
    E = logits.shape[1]
    last = K if K < E else E - 1
    if last == 0:
        return np.full(logits.shape[0], np.inf)
    gaps = srt[:, :last] - srt[:, 1:last + 1]
    return gaps.min(axis=1)


def screened_activations(w: wl.Workload, wr: torch.Tensor, bias: torch.Tensor, x: torch.Tensor = None,
                         max_attempts: int = 20):
    """X (CPU bf16) in which every token has a routing margin >= TAU; returns (x, n_redrawn)."""
    x = wl.activations(w, "cpu") if x is None else x.clone()
    wr_b, b = bits(wr), bias.cpu().numpy()
    redrawn = 0
    bad = np.arange(x.shape[0])
    for attempt in range(max_attempts):
        logits = oracle.route_logits(bits(x[torch.from_numpy(bad)]), wr_b, b)
        viol = bad[token_margins(logits, w.K) < TAU]
        if viol.size == 0:
            return x, redrawn
        x[torch.from_numpy(viol)] = wl.redraw_rows(w, int(viol.size), attempt, "cpu")
        redrawn += int(viol.size)
        bad = viol
    raise RuntimeError("could not build inputs with the routing margin")


def assert_close_rel_max(got: np.ndarray, ref: np.ndarray, what: str, rtol_of_max: float = FLOAT_RTOL_OF_MAX):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    scale = np.abs(ref).max() if ref.size else 0.0
    err = np.abs(got - ref).max() if ref.size else 0.0
    assert err <= rtol_of_max * scale + 1e-30, f"{what}: max|d| = {err:.3e} > {rtol_of_max} * {scale:.3e}"
    return err / scale if scale else 0.0


def predicted_histogram(w: wl.Workload, true_hist: np.ndarray, wr, bias) -> np.ndarray:
    """The workload's stand-in for the Distribution-Only predictor's output."""
    if w.prediction == "true":
        return np.asarray(true_hist, dtype=np.int32)
    if w.prediction == "noisy":
        return wl.noisy_prediction(w, torch.from_numpy(np.asarray(true_hist))).numpy()
    if w.prediction == "prev":
        xprev = wl.activations(w, "cpu", previous=True)
        idx, _, _ = oracle.route(bits(xprev), bits(wr), bias.cpu().numpy(), w.K, w.gate_mode)
        return oracle.histogram(idx, w.E).astype(np.int32)
    raise ValueError(w.prediction)
