// Warp-level epilogue of the router: top-K selection by warp shuffles and the gate weights.
#pragma once

#include <math_constants.h>

#include "common.cuh"

// One warp selects the K largest of `logit[0..E)` (shared memory, bias already added) in descending
// order, equal values by ascending index, and writes indices and gate weights of one token.
// Lane l owns experts l, l+32, ...; each of the K rounds is a warp arg-max by shuffles, after which
// the winner is struck from its owner's list.
template <int kMaxPerLane = 8>
__device__ __forceinline__ void warp_topk_gate(const float* logit, int E, int K, int gate_mode,
                                               int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
  const int lane = threadIdx.x & 31;
  float v[kMaxPerLane];
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) {
    const int e = lane + 32 * i;
    v[i] = e < E ? logit[e] : -CUDART_INF_F;
  }
  unsigned taken = 0;           // bit i: expert lane+32*i already selected
  float sel_v[8];
  int sel_e[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    sel_v[k] = 0.f;
    sel_e[k] = 0;
    if (k < K) {
      // local best: strict '>' keeps the lowest index among equal values
      float bv = -CUDART_INF_F;
      int be = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < kMaxPerLane; ++i) {
        const int e = lane + 32 * i;
        if (e < E && !((taken >> i) & 1u) && (be == 0x7fffffff || v[i] > bv)) {
          bv = v[i];
          be = e;
        }
      }
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, m);
        const int oe = __shfl_xor_sync(0xffffffffu, be, m);
        const bool other_valid = oe != 0x7fffffff, mine_valid = be != 0x7fffffff;
        if (other_valid && (!mine_valid || ov > bv || (ov == bv && oe < be))) {
          bv = ov;
          be = oe;
        }
      }
      sel_v[k] = bv;
      sel_e[k] = be;
      if ((be & 31) == lane) taken |= 1u << (be >> 5);
    }
  }
  if (lane == 0) {
    float g[8];
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      g[k] = 0.f;
      if (k < K) {
        // sel_v[0] is the largest logit
        g[k] = gate_mode == 0 ? __expf(sel_v[k] - sel_v[0]) : 1.f / (1.f + __expf(-sel_v[k]));
        sum += g[k];
      }
    }
    const float inv = 1.f / sum;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (k < K) {
        idx_out[k] = sel_e[k];
        w_out[k] = g[k] * inv;
      }
    }
  }
}
