// pack: Algorithm 1 of the paper itself - G devices with limited memory, several experts per device -
// on predicted per-expert token counts (Section 3.1; only proportions are known before routing,
// Section 3.2.1, so the dispatch is kept as counts share[e][g] = tokens of expert e served by device g).
//
// While max_g L_g - min_g L_g > 1: g_h = the most loaded device, g_c = the least loaded one (ties: the
// lowest device), Delta = ceil((L_gh - L_gc) / 2), e* = the expert with the most tokens on g_h (ties:
// the lowest expert) among those that g_c hosts already or may still receive (fewer than c_max copies
// and a free place on g_c); e* is copied to g_c if it is not there and min(Delta, share[e*][g_h]) of
// its tokens move from g_h to g_c.  The loop ends when the loads are within one token of each other or
// no expert of g_h can be served by g_c.  The algorithm is sequential by nature (each move depends
// on the loads the previous one left), so one warp runs it: lane l keeps the loads of devices l and
// l + 32 in registers, arg-max / arg-min and the choice of e* are shuffle butterflies over packed
// (value, index) keys, and the E x G share matrix lives in shared memory.  Integer only.
#include "common.cuh"

namespace {

constexpr int kMaxE = 256;
constexpr int kMaxG = 64;
constexpr int kMaxIters = 1 << 20;      // never reached: sum_g L_g^2 falls strictly with every move

__device__ __forceinline__ long long warp_max_ll(long long v) {
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    const long long o = __shfl_xor_sync(0xffffffffu, v, m);
    v = o > v ? o : v;
  }
  return v;
}

__global__ void __launch_bounds__(32)
pack_kernel(const int32_t* __restrict__ pred, const int32_t* __restrict__ home, const int32_t* __restrict__ capacity,
            int E, int G, int c_max, int32_t* __restrict__ placement, int32_t* __restrict__ share_out,
            int32_t* __restrict__ load_out, int32_t* __restrict__ iters_out, int32_t* __restrict__ status) {
  extern __shared__ int32_t share[];                 // [E][G]
  __shared__ unsigned long long placed[kMaxE];       // bit g: expert e has a copy on device g
  __shared__ int32_t copies[kMaxE];
  __shared__ int32_t used[kMaxG], cap[kMaxG];
  const int lane = threadIdx.x;

  for (int i = lane; i < E * G; i += 32) share[i] = 0;
  for (int g = lane; g < G; g += 32) { used[g] = 0; cap[g] = capacity[g]; }
  __syncwarp();
  bool bad = false;
  for (int e = lane; e < E; e += 32) {
    int h = home[e];
    int n = pred[e];
    if (h < 0 || h >= G || n < 0) {
      moegps_report(status, MOEGPS_ERR_BAD_INDEX, e);
      bad = true;
      h = h < 0 || h >= G ? 0 : h;
      n = n < 0 ? 0 : n;
    }
    placed[e] = 1ull << h;
    copies[e] = 1;
    share[e * G + h] = n;
    atomicAdd(&used[h], 1);
  }
  __syncwarp();
  for (int g = lane; g < G; g += 32)
    if (used[g] > cap[g]) { moegps_report(status, MOEGPS_ERR_BAD_INDEX, g); bad = true; }
  bad = __any_sync(0xffffffffu, bad);
  // loads of devices lane and lane + 32
  long long l0 = 0, l1 = 0;
  for (int e = 0; e < E; ++e) {
    if (lane < G) l0 += share[e * G + lane];
    if (lane + 32 < G) l1 += share[e * G + lane + 32];
  }
  {   // the loads are returned as int32: all predicted tokens together must fit
    long long total = l0 + l1;
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) total += __shfl_xor_sync(0xffffffffu, total, m);
    if (total > 0x7fffffffll) {
      if (lane == 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, E);
      bad = true;
    }
  }
  int iters = 0;
  while (!bad && iters < kMaxIters) {
    // (load, device) packed so that one max finds the hottest / coldest device, lowest index on ties
    const long long none = -1;
    long long hi = none, lo = none;
    if (lane < G) { hi = (l0 << 7) | (63 - lane); lo = (((1ll << 40) - l0) << 7) | (63 - lane); }
    if (lane + 32 < G) {
      const long long h1 = (l1 << 7) | (63 - (lane + 32)), c1 = (((1ll << 40) - l1) << 7) | (63 - (lane + 32));
      hi = h1 > hi ? h1 : hi;
      lo = c1 > lo ? c1 : lo;
    }
    hi = warp_max_ll(hi);
    lo = warp_max_ll(lo);
    const int g_h = 63 - (int)(hi & 127), g_c = 63 - (int)(lo & 127);
    const long long L_h = hi >> 7, L_c = (1ll << 40) - (lo >> 7);
    if (L_h - L_c <= 1) break;
    const long long delta = (L_h - L_c + 1) / 2;
    // e*: the biggest expert on g_h that g_c hosts or may receive (lowest index on ties)
    const bool room = used[g_c] < cap[g_c];
    long long best = none;
    for (int e = lane; e < E; e += 32) {
      const int s = share[e * G + g_h];
      if (s <= 0) continue;
      const bool there = (placed[e] >> g_c) & 1ull;
      if (there || (room && (c_max <= 0 || copies[e] < c_max))) {
        const long long key = ((long long)s << 9) | (511 - e);
        best = key > best ? key : best;
      }
    }
    best = warp_max_ll(best);
    if (best < 0) break;
    const int e_star = 511 - (int)(best & 511);
    const long long have = best >> 9;
    const long long m = delta < have ? delta : have;
    if (lane == 0) {
      if (!((placed[e_star] >> g_c) & 1ull)) {
        placed[e_star] |= 1ull << g_c;
        copies[e_star] += 1;
        used[g_c] += 1;
      }
      share[e_star * G + g_h] -= (int)m;
      share[e_star * G + g_c] += (int)m;
    }
    if (lane == (g_h & 31)) { if (g_h < 32) l0 -= m; else l1 -= m; }
    if (lane == (g_c & 31)) { if (g_c < 32) l0 += m; else l1 += m; }
    ++iters;
    __syncwarp();
  }
  if (iters >= kMaxIters && lane == 0) moegps_report(status, MOEGPS_ERR_TIMEOUT, iters);
  __syncwarp();
  for (int i = lane; i < E * G; i += 32) {
    share_out[i] = share[i];
    placement[i] = (int)((placed[i / G] >> (i % G)) & 1ull);
  }
  if (lane < G) load_out[lane] = (int32_t)l0;
  if (lane + 32 < G) load_out[lane + 32] = (int32_t)l1;
  if (lane == 0) iters_out[0] = iters;
}

// The placement as slot tables: one slot per (expert, device) copy, experts ascending and, within an
// expert, devices ascending; slots beyond the last copy are empty.  One CTA, thread e = expert e.
__global__ void __launch_bounds__(kMaxE)
pack_slots_kernel(const int32_t* __restrict__ placement, const int32_t* __restrict__ share, int E, int G, int S,
                  int32_t* __restrict__ replicas, int32_t* __restrict__ slot_off, int32_t* __restrict__ slot_expert,
                  int32_t* __restrict__ slot_share, int32_t* __restrict__ slot_device, int32_t* __restrict__ status) {
  __shared__ int warp_sum[kMaxE / 32];
  const int e = threadIdx.x, lane = e & 31, warp = e >> 5;
  int r = 0;
  if (e < E)
    for (int g = 0; g < G; ++g) r += placement[e * G + g] != 0;
  int incl = r;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  int base = 0, total = 0;
  for (int w = 0; w < kMaxE / 32; ++w) {
    if (w < warp) base += warp_sum[w];
    total += warp_sum[w];
  }
  const int first = base + incl - r;
  if (e == 0 && total > S) moegps_report(status, MOEGPS_ERR_BAD_INDEX, total);   // more copies than slots
  if (e < E) {
    replicas[e] = r;
    slot_off[e] = first;
    int s = first;
    for (int g = 0; g < G; ++g) {
      if (placement[e * G + g] != 0) {
        if (s < S) {
          slot_expert[s] = e;
          slot_share[s] = share[e * G + g];
          slot_device[s] = g;
        }
        ++s;
      }
    }
  }
  if (e == 0) slot_off[E] = total;
  for (int s = total + e; s < S; s += kMaxE) {
    slot_expert[s] = -1;
    slot_share[s] = 0;
    slot_device[s] = -1;
  }
}

bool ok16(const void* p) { return p != nullptr && moegps_aligned16(p); }

}  // namespace

extern "C" MOEGPS_API int moegps_pack_slots(moegps_ctx_t* ctx, const int32_t* placement, const int32_t* share,
                                            int32_t n_devices, int32_t* replicas, int32_t* slot_off,
                                            int32_t* slot_expert, int32_t* slot_share, int32_t* slot_device,
                                            void* stream) {
  if (!ctx || !ok16(placement) || !ok16(share) || !ok16(replicas) || !ok16(slot_off) || !ok16(slot_expert) ||
      !ok16(slot_share) || !ok16(slot_device))
    return MOEGPS_ERR_INVALID_ARG;
  if (n_devices < 1 || n_devices > kMaxG) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  if (int rc = moegps_check_device(ctx)) return rc;
  pack_slots_kernel<<<1, kMaxE, 0, (cudaStream_t)stream>>>(placement, share, ctx->shape.E, n_devices, ctx->shape.S,
                                                           replicas, slot_off, slot_expert, slot_share, slot_device,
                                                           ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

extern "C" MOEGPS_API int moegps_pack(moegps_ctx_t* ctx, const int32_t* predicted_hist, const int32_t* home,
                                      const int32_t* capacity, int32_t n_devices, int32_t* placement,
                                      int32_t* share, int32_t* load, int32_t* iterations, void* stream) {
  if (!ctx || !ok16(predicted_hist) || !ok16(home) || !ok16(capacity) || !ok16(placement) || !ok16(share) ||
      !ok16(load) || !iterations || (reinterpret_cast<uintptr_t>(iterations) & 3u))
    return MOEGPS_ERR_INVALID_ARG;
  if (n_devices < 1 || n_devices > kMaxG) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  if (int rc = moegps_check_device(ctx)) return rc;
  const int E = ctx->shape.E;
  const size_t smem = (size_t)E * n_devices * sizeof(int32_t);
  if (!ctx->pack_attr_done) {
    MOEGPS_CUDA_TRY(ctx, cudaFuncSetAttribute(pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kMaxE * kMaxG * (int)sizeof(int32_t)));
    ctx->pack_attr_done = true;
  }
  pack_kernel<<<1, 32, smem, (cudaStream_t)stream>>>(predicted_hist, home, capacity, E, n_devices, ctx->shape.c_max,
                                                     placement, share, load, iterations, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
