// plan: Algorithm 1 of the paper in slot form, on one CTA.  Warp 0 keeps (n_e, r_e) of all experts
// in registers (lane l: experts l, l+32, ...); each of the S-E rounds is an arg-max of n_e / r_e over
// the lanes' best candidates, which hands the next free slot to the winner.  The slot tables then
// come from a block scan.  Integer only.
//
// The rounds are a serial chain, so a round is kept short.  The ratio n/r is compared through the
// key floor(n 2^21 / r): r <= 1024, so two different ratios differ by at least 2^-20 and get
// different keys, equal ratios get equal keys - the order of the keys is exactly the order of the
// ratios (no rounding enters the choice), and a key costs two 32-bit divisions, paid only by the
// expert that has just won.  Ties go to fewer replicas, then to the lower index: a candidate is the
// 64-bit word (key << 11) | (2047 - r), larger first, and among equal words the lower expert.  A lane
// keeps the best of its own experts (it changes only when one of them wins); the warp-wide arg-max is
// three redux operations (high word, low word among those, expert index among those) instead of a
// shuffle butterfly.
#include "common.cuh"

namespace {

constexpr int kPlanThreads = 256;   // >= the largest supported E
constexpr uint32_t kNone = 0xffffffffu;

// Candidate word of an expert with count n (< 2^31) and r copies (1 <= r <= 1024): the ratio key
// floor(n 2^21 / r) (< 2^52) above 2047 - r.  0 = absent (r == 0) or at the copy limit: every real
// candidate is larger.
__device__ __forceinline__ unsigned long long candidate(uint32_t n, int r, int c_max) {
  if (r <= 0 || (c_max > 0 && r >= c_max)) return 0ull;
  const uint32_t ur = (uint32_t)r, q = n / ur, m = n - q * ur;
  const unsigned long long key = ((unsigned long long)q << 21) | (unsigned long long)((m << 21) / ur);
  return (key << 11) | (unsigned long long)(2047 - r);
}

// The S-E rounds on one warp, kPerLane experts per lane.  Returns the replica counts in plan_r.
template <int kPerLane>
__device__ __forceinline__ void plan_rounds(const int32_t* __restrict__ pred, int E, int S, int c_max, int* plan_r) {
  const int lane = threadIdx.x & 31;
  uint32_t ln[kPerLane];
  int lr[kPerLane];            // 0 = no such expert
  unsigned long long cand[kPerLane];
#pragma unroll
  for (int i = 0; i < kPerLane; ++i) {
    const int e = lane + 32 * i;
    const int v = e < E ? pred[e] : 0;
    ln[i] = v < 0 ? 0u : (uint32_t)v;
    lr[i] = e < E ? 1 : 0;
    cand[i] = candidate(ln[i], lr[i], c_max);
  }
  // the lane's best candidate and its position (the lowest position among equal words: a pairwise
  // tournament in which the right-hand side must be strictly larger to win)
  unsigned long long best;
  int best_i;
  auto lane_best = [&]() {
    unsigned long long c[kPerLane];
    int idx[kPerLane];
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) { c[i] = cand[i]; idx[i] = i; }
#pragma unroll
    for (int w = 1; w < kPerLane; w *= 2)
#pragma unroll
      for (int i = 0; i + w < kPerLane; i += 2 * w) {
        const bool take = c[i + w] > c[i];
        c[i] = take ? c[i + w] : c[i];
        idx[i] = take ? idx[i + w] : idx[i];
      }
    best = c[0];
    best_i = idx[0];
  };
  lane_best();
  for (int round = 0; round < S - E; ++round) {
    const uint32_t hi = (uint32_t)(best >> 32), lo = (uint32_t)best;
    const uint32_t hi_max = __reduce_max_sync(0xffffffffu, hi);
    const bool in1 = hi == hi_max;
    const uint32_t lo_max = __reduce_max_sync(0xffffffffu, in1 ? lo : 0u);
    const bool in2 = in1 && lo == lo_max && best != 0ull;
    const uint32_t e_win = __reduce_min_sync(0xffffffffu, in2 ? (uint32_t)(lane + 32 * best_i) : kNone);
    if (e_win == kNone) break;   // nobody may take another copy: the remaining slots stay empty
    if ((e_win & 31u) == (uint32_t)lane) {   // the winner's lane: one more copy, a new word, a new best
      uint32_t n_w = 0;
      int r_w = 0;
#pragma unroll
      for (int i = 0; i < kPerLane; ++i)
        if (i == best_i) { n_w = ln[i]; r_w = lr[i]; }
      r_w += 1;
      const unsigned long long c_w = candidate(n_w, r_w, c_max);
#pragma unroll
      for (int i = 0; i < kPerLane; ++i)
        if (i == best_i) { lr[i] = r_w; cand[i] = c_w; }
      lane_best();
    }
  }
#pragma unroll
  for (int i = 0; i < kPerLane; ++i)
    plan_r[lane + 32 * i] = lr[i];
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
  // The S-E rounds run on warp 0 alone (no block barriers inside the loop).
  if (warp == 0) {
    if (E <= 32) plan_rounds<1>(pred, E, S, c_max, plan_r);
    else if (E <= 64) plan_rounds<2>(pred, E, S, c_max, plan_r);
    else if (E <= 128) plan_rounds<4>(pred, E, S, c_max, plan_r);
    else plan_rounds<8>(pred, E, S, c_max, plan_r);
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
