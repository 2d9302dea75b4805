// Distribution-Only Prediction state on the device (paper, Section 3.2.1): the maximum-likelihood
// estimate p_e = n_e / N of Eq. 1 over all batches seen so far is kept as cumulative per-expert
// counts, i.e. Eq. 1 over the pooled tokens (the running average Section 3.2.1 describes for batched
// data), and the error rate |p_est - p| / (1/E) of Section 3.2.1, averaged over the experts as in
// Section 3.3, compares a prediction with what a batch did.
// Both are one-CTA kernels: E <= 256.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
predictor_update_kernel(const int32_t* __restrict__ hist, int E, long long* __restrict__ state,
                        int32_t* __restrict__ predicted, int32_t* __restrict__ status) {
  __shared__ long long warp_max[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  long long s = 0;
  if (tid < E) {
    const int h = hist[tid];
    if (h < 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, tid);
    s = state[tid] + (h < 0 ? 0 : h);
    state[tid] = s;
  }
  long long m = s;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  if (lane == 0) warp_max[warp] = m;
  __syncthreads();
  m = 0;
  for (int w = 0; w < kThreads / 32; ++w) m = max(m, warp_max[w]);
  // the plan only needs proportions: scale all counts down by the same power of two until the
  // largest fits an int32
  int shift = 0;
  while ((m >> shift) > 0x7fffffffll) ++shift;
  if (tid < E) predicted[tid] = (int32_t)(s >> shift);
}

// Exponentially weighted variant: the state holds counts in units of 2^-16 tokens and moves towards
// the new batch by floor((hist * 2^16 - state) / 2^shift), i.e. alpha = 2^-shift.  Integer only.
__global__ void __launch_bounds__(kThreads)
predictor_update_ema_kernel(const int32_t* __restrict__ hist, int E, int shift, long long* __restrict__ state,
                            int32_t* __restrict__ predicted, int32_t* __restrict__ status) {
  __shared__ long long warp_max[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  long long s = 0;
  if (tid < E) {
    int h = hist[tid];
    if (h < 0) {
      moegps_report(status, MOEGPS_ERR_BAD_INDEX, tid);
      h = 0;
    }
    const long long old = state[tid];
    s = old + ((((long long)h << 16) - old) >> shift);      // arithmetic shift = floor division
    state[tid] = s;
  }
  long long m = s;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  if (lane == 0) warp_max[warp] = m;
  __syncthreads();
  m = 0;
  for (int w = 0; w < kThreads / 32; ++w) m = max(m, warp_max[w]);
  int down = 0;
  while ((m >> down) > 0x7fffffffll) ++down;
  if (tid < E) predicted[tid] = (int32_t)(s >> down);
}

__global__ void __launch_bounds__(kThreads)
error_rate_kernel(const int32_t* __restrict__ predicted, const int32_t* __restrict__ hist, int E,
                  double* __restrict__ out) {
  __shared__ long long warp_a[kThreads / 32], warp_b[kThreads / 32];
  __shared__ double warp_d[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long a = tid < E ? predicted[tid] : 0, b = tid < E ? hist[tid] : 0;
  long long sa = a, sb = b;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    sa += __shfl_xor_sync(0xffffffffu, sa, d);
    sb += __shfl_xor_sync(0xffffffffu, sb, d);
  }
  if (lane == 0) { warp_a[warp] = sa; warp_b[warp] = sb; }
  __syncthreads();
  long long ta = 0, tb = 0;
  for (int w = 0; w < kThreads / 32; ++w) { ta += warp_a[w]; tb += warp_b[w]; }
  // |p_est - p| in units of 1/E, then the mean over the experts: E * |..| / E = |..| summed
  double diff = 0.0;
  if (tid < E && ta > 0 && tb > 0) diff = fabs((double)a / (double)ta - (double)b / (double)tb);
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) diff += __shfl_xor_sync(0xffffffffu, diff, d);   // fixed order: deterministic
  if (lane == 0) warp_d[warp] = diff;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) t += warp_d[w];
    out[0] = (ta > 0 && tb > 0) ? t : 0.0;
  }
}

bool ok16(const void* p) { return p != nullptr && moegps_aligned16(p); }

}  // namespace

extern "C" MOEGPS_API int moegps_predictor_update(moegps_ctx_t* ctx, const int32_t* hist, int64_t* state,
                                                  int32_t* predicted_hist, void* stream) {
  if (!ctx || !ok16(hist) || !ok16(state) || !ok16(predicted_hist)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  predictor_update_kernel<<<1, kThreads, 0, (cudaStream_t)stream>>>(hist, ctx->shape.E,
                                                                     reinterpret_cast<long long*>(state),
                                                                     predicted_hist, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

extern "C" MOEGPS_API int moegps_predictor_update_ema(moegps_ctx_t* ctx, const int32_t* hist, int64_t* state,
                                                      int32_t shift, int32_t* predicted_hist, void* stream) {
  if (!ctx || !ok16(hist) || !ok16(state) || !ok16(predicted_hist) || shift < 0 || shift > 16)
    return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  predictor_update_ema_kernel<<<1, kThreads, 0, (cudaStream_t)stream>>>(
      hist, ctx->shape.E, shift, reinterpret_cast<long long*>(state), predicted_hist, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

extern "C" MOEGPS_API int moegps_error_rate(moegps_ctx_t* ctx, const int32_t* predicted_hist, const int32_t* hist,
                                            double* error_rate, void* stream) {
  if (!ctx || !ok16(predicted_hist) || !ok16(hist) || !error_rate ||
      (reinterpret_cast<uintptr_t>(error_rate) & 7u))
    return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  error_rate_kernel<<<1, kThreads, 0, (cudaStream_t)stream>>>(predicted_hist, hist, ctx->shape.E, error_rate);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
