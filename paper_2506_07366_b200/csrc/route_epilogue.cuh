// Warp-level epilogue of the router: top-K selection by shuffles inside groups of lanes and the gate
// weights.
#pragma once

#include <math_constants.h>

#include "common.cuh"

// Monotone map from fp32 to uint32 (larger float <=> larger key); -0 is folded into +0 first so
// that equal values have equal keys.  No finite float maps to key 0, which marks "no candidate".
__device__ __forceinline__ uint32_t route_order_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float route_key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// L lanes per token (L = 4, 8, 16 or 32; a warp works on 32/L tokens at once; every lane of the warp
// must call this).  Sub-lane l holds the order keys of experts l, l+L, ... in key[0..NPL) (0 = no
// such expert).  Each of the K rounds: every lane finds its best remaining entry (strict '>' in
// ascending index keeps the lowest index among equal keys), a log2(L)-step xor butterfly over
// (key, index) - larger key first, lower index among equal keys - leaves the group's winner in all
// L lanes, and its owner strikes it.  Selections come out in descending logit order, equal logits by
// ascending expert index.  Then sub-lane k < K computes the k-th gate weight (mode 0: softmax over
// the selected K; mode 1: sigmoid, renormalised over the selected K) and, if `store`, writes index
// and weight.  Returns the expert this lane holds (sub-lane k < K: the k-th selection), else -1.
// Requires K <= L.  Why lane groups and plain shuffles: measured on B200 against one token per warp
// with two redux.sync per round, groups of eight shorten the selection phase of a tile by 1.3-2x
// (E = 8 .. 64); redux.sync cost 100-350 cycles per operation there with twelve warps in flight.
// The caller picks L so that the rows a CTA owns occupy all its warps in one pass.
template <int L, int NPL>
__device__ __forceinline__ int group_topk_gate(uint32_t (&key)[NPL], int K, int gate_mode, bool store,
                                               int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
  const int sl = threadIdx.x & (L - 1);
  float myv = 0.f, top_v = 0.f;   // this sub-lane's selection (the sl-th) and the largest logit
  int mye = 0;
  // The rounds stay a loop (not unrolled): the kernel runs once per layer with cold instruction
  // caches, and fetching K copies of the scan below costs more than the loop overhead saves.
#pragma unroll 1
  for (int k = 0; k < K; ++k) {
    uint32_t bk = 0u;
    int be = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < NPL; ++i) {
      if (key[i] > bk) {
        bk = key[i];
        be = sl + L * i;
      }
    }
#pragma unroll
    for (int m = 1; m < L; m <<= 1) {
      const uint32_t ok = __shfl_xor_sync(0xffffffffu, bk, m);
      const int oe = __shfl_xor_sync(0xffffffffu, be, m);
      if (ok > bk || (ok == bk && oe < be)) {
        bk = ok;
        be = oe;
      }
    }
    const float v = route_key_value(bk);
    if (k == 0) top_v = v;
    if (k == sl) {
      myv = v;
      mye = be;
    }
#pragma unroll
    for (int i = 0; i < NPL; ++i)
      if (be == sl + L * i) key[i] = 0u;
  }
  float g = 0.f;
  if (sl < K) g = gate_mode == 0 ? __expf(myv - top_v)
                                 : 1.f / (1.f + __expf(-myv));
  float sum = g;                 // sub-lanes K..L-1 contribute 0
#pragma unroll
  for (int m = 1; m < L; m <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
  if (store && sl < K) {
    idx_out[sl] = mye;
    w_out[sl] = g / sum;
  }
  return sl < K ? mye : -1;
}
