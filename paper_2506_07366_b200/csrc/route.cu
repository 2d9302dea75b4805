// route: router GEMM fused with bias, warp-shuffle top-K and the gate weights (paper, Section 2).
// One warp per token: the lanes split the model dimension (128-bit loads of X and of the router
// rows), partial dot products are reduced by shuffles into a per-warp logit row in shared memory,
// and the warp then selects the K largest logits (route_epilogue.cuh).
#include "common.cuh"
#include "route_epilogue.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kMaxE = 256;
constexpr int kEG = 8;     // experts per pass over the token row

__device__ __forceinline__ void dot8(float& acc, const uint4& a, const uint4& b) {
  const uint32_t ua[4] = {a.x, a.y, a.z, a.w}, ub[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc = fmaf(__uint_as_float(ua[i] << 16), __uint_as_float(ub[i] << 16), acc);
    acc = fmaf(__uint_as_float(ua[i] & 0xffff0000u), __uint_as_float(ub[i] & 0xffff0000u), acc);
  }
}

__global__ void __launch_bounds__(kThreads)
route_kernel(const uint4* __restrict__ x, const uint4* __restrict__ wr, const float* __restrict__ bias, int T,
             int chunks /* D/8 */, int E, int K, int gate_mode, int32_t* __restrict__ topk_idx,
             float* __restrict__ topk_w, float* __restrict__ logits_out) {
  __shared__ float logit[kWarpsPerBlock][kMaxE];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= T) return;
  const uint4* xr = x + (int64_t)t * chunks;
  for (int e0 = 0; e0 < E; e0 += kEG) {
    float acc[kEG];
#pragma unroll
    for (int i = 0; i < kEG; ++i) acc[i] = 0.f;
    for (int c = lane; c < chunks; c += 32) {
      const uint4 xv = xr[c];
#pragma unroll
      for (int i = 0; i < kEG; ++i)
        if (e0 + i < E) dot8(acc[i], xv, wr[(int64_t)(e0 + i) * chunks + c]);
    }
#pragma unroll
    for (int i = 0; i < kEG; ++i) {
      float v = acc[i];
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
      if (lane == 0 && e0 + i < E) logit[warp][e0 + i] = v + (bias ? bias[e0 + i] : 0.f);
    }
  }
  __syncwarp();
  if (logits_out) {
    for (int e = lane; e < E; e += 32) logits_out[(int64_t)t * E + e] = logit[warp][e];
    if (!topk_idx) return;
  }
  warp_topk_gate<kMaxE / 32>(logit[warp], E, K, gate_mode, topk_idx + (int64_t)t * K, topk_w + (int64_t)t * K);
}

}  // namespace

int moegps_launch_route(moegps_ctx* ctx, const void* x, const void* wr, const float* bias, int32_t* topk_idx,
                        float* topk_w, float* logits_out, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int blocks = (s.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  route_kernel<<<blocks, kThreads, 0, st>>>(static_cast<const uint4*>(x), static_cast<const uint4*>(wr), bias, s.T,
                                            s.D / 8, s.E, s.K, s.gate_mode, topk_idx, topk_w, logits_out);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
