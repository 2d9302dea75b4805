"""Seeded synthetic inputs for the MoE hot path.

This module only draws random tensors of stated shapes and distributions; it holds none of the
method's arithmetic (no routing, counting, planning or expert math) and imports neither the CUDA
binding nor the CPU oracle, so both sides of a parity test can be fed from it.

The five workloads stand in for the paper's measurements on Mixtral-8x7B activations (Section
3.2.1: sequence length 512, skewness 1.39-1.99) and its many-expert discussion: the layer shapes
are Mixtral's (4096 x 14336, 8 experts, top-2) and two finer-grained expert layouts; the skew comes
from a per-expert router bias with Zipf-like masses.  Datasets and trained weights are not used.

Recipe
  expert weights  W1, W3 [E, F, D], W2 [E, D, F]  ~ N(0, 0.02^2), bf16
  activations     X [T, D] ~ N(0, sigma_x^2), bf16   (sigma_x = 0.02 for "tiny", else 1)
  router          Wr [E, D] ~ N(0, sigma_r^2), sigma_r = 1 / (sigma_x sqrt(D))  => unit-variance logits
  router bias     b_e = -s * ln(rank_e), rank a seeded permutation of 1..E (log of a Zipf(s) mass)
  prediction      "prev": histogram of a previous batch (drawn from stream +7);
                  "true": the batch's own histogram;
                  "noisy": round(max(0, n_e * (1 + 0.1 z_e))), z ~ N(0, 1) from stream +6
Seeds: base 250607366 + 1000 * (config number); sub-streams +0 X, +1 Wr, +2 rank permutation,
+3/+4/+5 W1/W3/W2, +6 prediction noise, +7 previous-batch X, +8 re-draws of X rows.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    number: int          # 1-based position in the list of workloads (seeds derive from it)
    T: int
    D: int
    F: int
    E: int
    K: int
    S: int
    gate_mode: int       # 0 softmax over the selected experts, 1 sigmoid then renormalise
    zipf_s: float
    sigma_x: float
    prediction: str      # "prev" | "true" | "noisy"

    @property
    def R(self) -> int:
        return self.T * self.K

    @property
    def seed(self) -> int:
        return 250607366 + 1000 * self.number

    def scaled(self, **kw) -> "Workload":
        """Same recipe at other sizes (used for parity cases the oracle finishes quickly)."""
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    "tiny": Workload("tiny", 1, T=256, D=512, F=1024, E=8, K=2, S=8, gate_mode=0,
                     zipf_s=1.0, sigma_x=0.02, prediction="prev"),
    "mixtral": Workload("mixtral", 2, T=4096, D=4096, F=14336, E=8, K=2, S=8, gate_mode=0,
                        zipf_s=0.8, sigma_x=1.0, prediction="true"),
    "mixtral_skew": Workload("mixtral_skew", 3, T=16384, D=4096, F=14336, E=8, K=2, S=16,
                             gate_mode=0, zipf_s=1.5, sigma_x=1.0, prediction="noisy"),
    "many_expert": Workload("many_expert", 4, T=8192, D=2048, F=1408, E=64, K=6, S=80,
                            gate_mode=0, zipf_s=1.2, sigma_x=1.0, prediction="noisy"),
    "fine_grained": Workload("fine_grained", 5, T=4096, D=7168, F=2048, E=256, K=8, S=288,
                             gate_mode=1, zipf_s=1.0, sigma_x=1.0, prediction="noisy"),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _normal_bf16(shape, std: float, seed: int, device) -> torch.Tensor:
    """bf16 N(0, std^2).  Drawn in fp32 chunk by chunk along the first axis so that very large
    tensors never need an fp32 copy of themselves."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    g = _gen(seed, device)
    n0 = shape[0]
    per = max(1, int(math.prod(shape[1:])))
    step = max(1, (1 << 26) // per)
    for lo in range(0, n0, step):
        hi = min(n0, lo + step)
        chunk = torch.randn((hi - lo,) + tuple(shape[1:]), generator=g, device=device,
                            dtype=torch.float32)
        out[lo:hi] = (chunk * std).to(torch.bfloat16)
    return out


def activations(w: Workload, device="cpu", previous: bool = False) -> torch.Tensor:
    """X [T, D] bf16; `previous` draws the batch that precedes it (stream +7)."""
    return _normal_bf16((w.T, w.D), w.sigma_x, w.seed + (7 if previous else 0), device)


def redraw_rows(w: Workload, n_rows: int, attempt: int, device="cpu") -> torch.Tensor:
    """Fresh rows of X from stream +8, for callers that replace rows (e.g. near-tied tokens)."""
    return _normal_bf16((n_rows, w.D), w.sigma_x, w.seed + 8 + 100 * (attempt + 1), device)


def router(w: Workload, device="cpu"):
    """(Wr [E, D] bf16, bias [E] fp32)."""
    sigma_r = 1.0 / (w.sigma_x * math.sqrt(w.D))
    wr = _normal_bf16((w.E, w.D), sigma_r, w.seed + 1, device)
    g = _gen(w.seed + 2, "cpu")
    rank = torch.randperm(w.E, generator=g) + 1
    bias = (-w.zipf_s * torch.log(rank.to(torch.float64))).to(torch.float32)
    return wr, bias.to(device)


def expert_weights(w: Workload, device="cpu"):
    """(W1 [E, F, D], W3 [E, F, D], W2 [E, D, F]) bf16 ~ N(0, 0.02^2)."""
    w1 = _normal_bf16((w.E, w.F, w.D), 0.02, w.seed + 3, device)
    w3 = _normal_bf16((w.E, w.F, w.D), 0.02, w.seed + 4, device)
    w2 = _normal_bf16((w.E, w.D, w.F), 0.02, w.seed + 5, device)
    return w1, w3, w2


def noisy_prediction(w: Workload, hist: torch.Tensor) -> torch.Tensor:
    """A histogram with 10 % seeded multiplicative noise: round(max(0, n_e (1 + 0.1 z_e)))."""
    g = _gen(w.seed + 6, "cpu")
    z = torch.randn(w.E, generator=g, dtype=torch.float64)
    h = hist.detach().to("cpu", torch.float64)
    return torch.clamp(torch.round(h * (1.0 + 0.1 * z)), min=0).to(torch.int32)


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view of a bf16 tensor's bits (host copy)."""
    import numpy as np
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)
