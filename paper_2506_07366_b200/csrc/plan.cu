// plan: Algorithm 1 of the paper in slot form, on one CTA.  Warp 0 keeps (n_e, r_e) of all experts
// in registers (lane l: experts l, l+32, ...); each of the S-E rounds is an arg-max of n_e / r_e
// (exact: 64-bit cross-multiplication) over the lanes' best candidates by a shuffle butterfly, which
// hands the next free slot to the winner.  The slot tables then come from a block scan.  Integer only.
#include "common.cuh"

namespace {

constexpr int kPlanThreads = 256;   // >= the largest supported E

// A candidate in two 32-bit registers (the rounds are a chain of shuffles, so every register
// counts): n = predicted count, re = (replicas << 12) | expert, kNone = not eligible.
// (replicas <= 1024 and expert < 288 fit 11 + 12 bits; comparing `re` compares replicas first,
// then the expert index - exactly the order in which equal ratios are resolved.)
struct Cand {
  uint32_t n;
  uint32_t re;
};
constexpr uint32_t kNone = 0xffffffffu;

// Strict order of Algorithm 1's choice: larger n/r first (exact: 64-bit cross-multiplication),
// then fewer replicas, then lower index.
__device__ __forceinline__ bool better(const Cand& a, const Cand& b) {
  if (a.re == kNone) return false;
  if (b.re == kNone) return true;
  const unsigned long long lhs = (unsigned long long)a.n * (b.re >> 12);
  const unsigned long long rhs = (unsigned long long)b.n * (a.re >> 12);
  if (lhs != rhs) return lhs > rhs;
  return a.re < b.re;
}

__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    Cand o;
    o.n = __shfl_xor_sync(0xffffffffu, c.n, m);
    o.re = __shfl_xor_sync(0xffffffffu, c.re, m);
    if (better(o, c)) c = o;
  }
  return c;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t* __restrict__ pred, int E, int S, int c_max, int32_t* __restrict__ replicas,
            int32_t* __restrict__ slot_off, int32_t* __restrict__ slot_expert, int32_t* __restrict__ bound,
            int32_t* __restrict__ status) {
  __shared__ int plan_r[kPlanThreads];
  __shared__ int warp_sum[kPlanThreads / 32];
  __shared__ int warp_max[kPlanThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool mine = tid < E;
  long long n = -1;
  int r = 0;
  if (mine) {
    const int v = pred[tid];
    if (v < 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, tid);
    n = v < 0 ? 0 : v;
    r = 1;
  }
  // The S-E rounds run on warp 0 alone (no block barriers inside the loop): lane l keeps experts
  // l, l+32, ... in registers, picks its best candidate, and a shuffle butterfly picks the winner.
  if (warp == 0) {
    constexpr int kPerLane = kPlanThreads / 32;
    uint32_t ln[kPerLane];
    int lr[kPerLane];            // 0 = no such expert
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
      const int e = lane + 32 * i;
      const int v = e < E ? pred[e] : 0;
      ln[i] = v < 0 ? 0u : (uint32_t)v;
      lr[i] = e < E ? 1 : 0;
    }
    for (int round = 0; round < S - E; ++round) {
      Cand c;
      c.n = 0; c.re = kNone;
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        Cand d;
        d.n = ln[i];
        d.re = (lr[i] > 0 && (c_max <= 0 || lr[i] < c_max)) ? (((uint32_t)lr[i] << 12) | (uint32_t)(lane + 32 * i))
                                                            : kNone;
        if (better(d, c)) c = d;
      }
      c = warp_best(c);
      if (c.re == kNone) break;    // nobody may take another copy: the remaining slots stay empty
      const int win = (int)(c.re & 0xfffu);
#pragma unroll
      for (int i = 0; i < kPerLane; ++i)
        if (win == lane + 32 * i) lr[i] += 1;
    }
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) plan_r[lane + 32 * i] = lr[i];
  }
  __syncthreads();
  if (mine) r = plan_r[tid];
  // slot_off = exclusive prefix sum of r
  int incl = mine ? r : 0;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_sum[warp] = incl;
  int b = mine ? (int)((n + r - 1) / r) : 0;     // ceil(n_e / r_e)
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) b = max(b, __shfl_xor_sync(0xffffffffu, b, m));
  if (lane == 0) warp_max[warp] = b;
  __syncthreads();
  int base = 0, total = 0, bmax = 0;
  for (int wv = 0; wv < kPlanThreads / 32; ++wv) {
    if (wv < warp) base += warp_sum[wv];
    total += warp_sum[wv];
    bmax = max(bmax, warp_max[wv]);
  }
  const int excl = base + incl - (mine ? r : 0);
  if (mine) {
    replicas[tid] = r;
    slot_off[tid] = excl;
    for (int s = excl; s < excl + r; ++s) slot_expert[s] = tid;
  }
  if (tid == 0) {
    slot_off[E] = total;
    bound[0] = bmax;
  }
  for (int s = total + tid; s < S; s += kPlanThreads) slot_expert[s] = -1;
}

}  // namespace

int moegps_launch_plan(moegps_ctx* ctx, const int32_t* pred, int32_t* replicas, int32_t* slot_off,
                       int32_t* slot_expert, int32_t* bound, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  plan_kernel<<<1, kPlanThreads, 0, st>>>(pred, s.E, s.S, s.c_max, replicas, slot_off, slot_expert, bound,
                                          ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
