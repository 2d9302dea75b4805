// Slot row offsets of the dispatch step (shared by the three dispatch kernels that derive them):
// how an expert's pairs are split over its copies, the rows each slot reserves, and their prefix sum.
#pragma once

#include "common.cuh"

namespace slot_offsets {

constexpr int kMaxS = 1024;

// Total of the predicted tokens that the copies of an expert were given (slot_share, from
// moegps_pack_slots); 0 when there is no share table, the prediction gave the expert nothing, or the
// table is out of range (then the copies take equal parts).
__device__ __forceinline__ long long share_total(const int32_t* __restrict__ slot_share, int so, int r) {
  if (!slot_share) return 0;
  long long tot = 0;
  for (int rho = 0; rho < r; ++rho) {
    const int v = slot_share[so + rho];
    if (v < 0) return 0;
    tot += v;
  }
  return tot > 0x7fffffffll ? 0 : tot;
}

// Rows reserved for the replicas of expert `e` (loads rounded up to A) -> padded[slot].
// Replica rho takes ranks floor(rho n/r) .. floor((rho+1) n/r) - 1, or, with a share table, ranks
// floor(n c_rho / c) .. floor(n c_{rho+1} / c) - 1 with c_rho the shares of the copies before it.
__device__ __forceinline__ void slot_loads_of_expert(int e, int S, int A, const int32_t* __restrict__ hist,
                                                     const int32_t* __restrict__ replicas,
                                                     const int32_t* __restrict__ slot_off,
                                                     const int32_t* __restrict__ slot_share, int32_t* padded,
                                                     int32_t* status) {
  const long long n = hist[e];
  const int r = replicas[e];
  const int so = slot_off[e];
  if (r < 1 || so < 0 || so + r > S || n < 0) {
    moegps_report(status, MOEGPS_ERR_BAD_INDEX, e);
    return;
  }
  const long long tot = share_total(slot_share, so, r);
  if (tot > 0) {
    long long cum = 0;
    int prev = 0;
    for (int rho = 0; rho < r; ++rho) {
      cum += slot_share[so + rho];
      const int start = (int)((n * cum) / tot);      // n, cum < 2^31
      padded[so + rho] = (start - prev + A - 1) / A * A;
      prev = start;
    }
    return;
  }
  // floor(rho n / r) = rho q + floor(rho m / r) with n = q r + m: one division, then 32-bit work
  const int q = (int)(n / r), m = (int)(n - (long long)q * r);
  int prev = 0;
  for (int rho = 1; rho <= r; ++rho) {
    const int start = rho * q + (rho * m) / r;     // rho, m < r <= 1024
    padded[so + rho - 1] = (start - prev + A - 1) / A * A;
    prev = start;
  }
}

// slot_row_off[0..S] for one thread block of kBlock threads (all of them must call; uses
// __syncthreads): padded[] (shared, kMaxS ints) receives the rows each slot reserves, then the
// offsets are their prefix sum - slot starts are multiples of A, so no further rounding is needed.
// Thread t owns slots kPer*t .. kPer*t + kPer-1.
template <int kBlock>
__device__ __forceinline__ void build_slot_row_off(int E, int S, int A, const int32_t* __restrict__ hist,
                                                   const int32_t* __restrict__ replicas,
                                                   const int32_t* __restrict__ slot_off,
                                                   const int32_t* __restrict__ slot_share, int32_t* padded,
                                                   int32_t* warp_tot /* shared, kBlock/32 ints */,
                                                   int32_t* __restrict__ slot_row_off, int32_t* status) {
  static_assert(kBlock % 32 == 0 && kBlock <= 1024, "whole warps");
  constexpr int kPer = (kMaxS + kBlock - 1) / kBlock;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int s = tid; s < S; s += kBlock) padded[s] = 0;
  __syncthreads();
  for (int e = tid; e < E; e += kBlock) slot_loads_of_expert(e, S, A, hist, replicas, slot_off, slot_share, padded, status);
  __syncthreads();
  int v[kPer], sum = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int s = kPer * tid + i;
    v[i] = s < S ? padded[s] : 0;
    sum += v[i];
  }
  int incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int run = incl - sum;
  for (int wv = 0; wv < warp; ++wv) run += warp_tot[wv];
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int s = kPer * tid + i;
    run += v[i];
    if (s < S) slot_row_off[s + 1] = run;
  }
  if (tid == 0) slot_row_off[0] = 0;
}

}  // namespace slot_offsets
