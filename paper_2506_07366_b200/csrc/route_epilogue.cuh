// Warp-level epilogue of the router: top-K selection across the lanes of a warp and the gate weights.
#pragma once

#include <math_constants.h>

#include "common.cuh"

// Monotone map from fp32 to uint32 (larger float <=> larger key); -0 is folded into +0 first so
// that equal values have equal keys.
__device__ __forceinline__ uint32_t route_order_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float route_key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// A group of G lanes (G = 8, 16 or 32; a warp holds 32/G independent groups, one token each) selects
// the K largest of E logits, in descending order, equal values by ascending expert index; sub-lane
// k < K of the group writes the k-th index and gate weight.  Sub-lane l holds the logits of experts
// l, l+G, ... in v[0..NPL) (NPL > 1 only with G = 32).  Each of the K rounds: every lane finds its
// best remaining entry, a max-reduction over the group (redux.sync with the group's lane mask) finds
// the winning value, a min-reduction over the lanes that hold it finds the lowest such expert, and
// its owner strikes it from its list.  Requires K <= 8 <= G.
template <int NPL, int G>
__device__ __forceinline__ void group_topk_gate(const float (&v)[NPL], int E, int K, int gate_mode,
                                                int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
  static_assert(G == 32 || NPL == 1, "several experts per lane only with whole-warp groups");
  const int lane = threadIdx.x & 31;
  const int sl = lane & (G - 1);
  const unsigned gmask = G == 32 ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(G - 1)));
  uint32_t key[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) key[i] = (sl + G * i < E) ? route_order_key(v[i]) : 0u;   // 0 < every real key
  unsigned taken = 0;           // bit i: expert sl+G*i already selected
  float sel_v[8];
  int sel_e[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    sel_v[k] = 0.f;
    sel_e[k] = 0;
    if (k < K) {
      uint32_t bk = 0u;         // best remaining key of this lane; strict '>' keeps its lowest index
      int be = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < NPL; ++i) {
        const bool live = (sl + G * i < E) && !((taken >> i) & 1u);
        if (live && (be == 0x7fffffff || key[i] > bk)) {
          bk = key[i];
          be = sl + G * i;
        }
      }
      const uint32_t wk = __reduce_max_sync(gmask, be == 0x7fffffff ? 0u : bk);
      const uint32_t we = __reduce_min_sync(gmask, (be != 0x7fffffff && bk == wk) ? (uint32_t)be : 0xffffffffu);
      sel_v[k] = route_key_value(wk);
      sel_e[k] = (int)we;
      if ((int)(we & (G - 1)) == sl) taken |= 1u << (we / G);
    }
  }
  // every lane knows all K selections; sub-lane k < K computes and stores the k-th gate weight
  float myv = 0.f;
  int mye = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    if (k < K && sl == k) {
      myv = sel_v[k];
      mye = sel_e[k];
    }
  }
  float g = 0.f;
  if (sl < K) g = gate_mode == 0 ? __expf(myv - sel_v[0]) /* sel_v[0] is the largest logit */
                                 : 1.f / (1.f + __expf(-myv));
  float sum = g;                 // sub-lanes K..7 contribute 0; the xor pattern stays inside 8 lanes
  sum += __shfl_xor_sync(gmask, sum, 1);
  sum += __shfl_xor_sync(gmask, sum, 2);
  sum += __shfl_xor_sync(gmask, sum, 4);
  if (sl < K) {
    idx_out[sl] = mye;
    w_out[sl] = g / sum;
  }
}
