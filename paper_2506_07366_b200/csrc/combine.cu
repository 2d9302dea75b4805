// combine: the post-FFN shuffle back to token order (paper, Section 2), as a gather:
//   out[t,:] = sum_{j<K} topk_w[t,j] * yp[pair_row[t,j],:]
// One warp per token, 128-bit loads of the K expert rows, fp32 accumulation in ascending j,
// bf16 round-to-nearest-even on store.  No atomics => deterministic.
#include "common.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;

__device__ __forceinline__ void fma8(float (&acc)[8], float w, const uint4& v) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // a bf16 is the upper half of an fp32
    acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
    acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
  }
}

__device__ __forceinline__ uint4 pack8(const float (&acc)[8]) {
  uint32_t u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    u[i] = *reinterpret_cast<const uint32_t*>(&h);
  }
  return make_uint4(u[0], u[1], u[2], u[3]);
}

template <int KT>   // KT = compile-time K (1..8)
__global__ void __launch_bounds__(kThreads)
combine_kernel(const uint4* __restrict__ yp, const int32_t* __restrict__ pair_row,
               const float* __restrict__ topk_w, int T, int chunks, int64_t Rcap, uint4* __restrict__ out,
               int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= T) return;
  const uint4* src[KT];
  float w[KT];
#pragma unroll
  for (int j = 0; j < KT; ++j) {
    int row = pair_row[(int64_t)t * KT + j];
    w[j] = topk_w[(int64_t)t * KT + j];
    if (row < 0 || row >= Rcap) {
      if (lane == 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, t);
      row = 0;
      w[j] = 0.f;
    }
    src[j] = yp + (int64_t)row * chunks;
  }
  uint4* dst = out + (int64_t)t * chunks;
  int c = lane;
  for (; c + 32 < chunks; c += 64) {        // 2*KT loads in flight per lane
    uint4 va[KT], vb[KT];
#pragma unroll
    for (int j = 0; j < KT; ++j) { va[j] = src[j][c]; vb[j] = src[j][c + 32]; }
    float a[8] = {0, 0, 0, 0, 0, 0, 0, 0}, b[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < KT; ++j) { fma8(a, w[j], va[j]); fma8(b, w[j], vb[j]); }
    dst[c] = pack8(a);
    dst[c + 32] = pack8(b);
  }
  for (; c < chunks; c += 32) {
    float a[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < KT; ++j) fma8(a, w[j], src[j][c]);
    dst[c] = pack8(a);
  }
}

}  // namespace

int moegps_launch_combine(moegps_ctx* ctx, const void* yp, const int32_t* pair_row, const float* topk_w,
                          void* out, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int blocks = (s.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  const int chunks = s.D / 8;
  const int64_t Rcap = moegps_rcap_of(s);
  const uint4* y = static_cast<const uint4*>(yp);
  uint4* o = static_cast<uint4*>(out);
#define MOEGPS_COMBINE_CASE(KT)                                                                           \
  case KT:                                                                                                \
    combine_kernel<KT><<<blocks, kThreads, 0, st>>>(y, pair_row, topk_w, s.T, chunks, Rcap, o, ctx->d_status); \
    break;
  switch (s.K) {
    MOEGPS_COMBINE_CASE(1) MOEGPS_COMBINE_CASE(2) MOEGPS_COMBINE_CASE(3) MOEGPS_COMBINE_CASE(4)
    MOEGPS_COMBINE_CASE(5) MOEGPS_COMBINE_CASE(6) MOEGPS_COMBINE_CASE(7) MOEGPS_COMBINE_CASE(8)
    default: return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  }
#undef MOEGPS_COMBINE_CASE
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
