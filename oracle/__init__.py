"""CPU oracle for the MoE hot path (route, histogram, plan, dispatch, expert_ffn, combine).

This package is TEST INFRASTRUCTURE.  It is a slow, plain numpy/fp64 statement of what each
step computes, written from the paper's definitions, and it is the yardstick the CUDA kernels
are compared with.  It shares no code with the CUDA path and must never be imported by the
product package; only the test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
"""
from .moe_oracle import (  # noqa: F401
    bf16_bits_to_f64,
    route_logits,
    route,
    histogram,
    p_hat,
    skewness,
    error_rate,
    predictor_update,
    predictor_update_ema,
    plan,
    pack,
    pack_slots,
    replica_starts,
    replica_starts_by_share,
    dispatch,
    expert_ffn,
    combine,
    moe_layer,
)
