// histogram: n_e = number of routed pairs whose expert is e (Eq. 1 of the paper with N = T*K).
// Shared-memory privatised counters, one warp-aggregated shared atomic per distinct expert a warp
// sees in a round, one global atomic per (CTA, expert).  Integer atomics only => deterministic.
#include "common.cuh"

namespace {

constexpr int kHistThreads = 256;

__global__ void __launch_bounds__(kHistThreads)
histogram_kernel(const int32_t* __restrict__ topk_idx, int64_t R, int E, int32_t* __restrict__ hist,
                 int32_t* __restrict__ status) {
  __shared__ int32_t cnt[256];
  for (int e = threadIdx.x; e < E; e += blockDim.x) cnt[e] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  // every warp iterates the same number of rounds so that the match below is warp-uniform
  const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t rounds = (R + stride - 1) / stride;
  for (int64_t it = 0; it < rounds; ++it) {
    const int64_t p = first + it * stride;
    int e = -1;
    if (p < R) {
      e = topk_idx[p];
      if (e < 0 || e >= E) {
        moegps_report(status, MOEGPS_ERR_BAD_INDEX, (int)(p & 0x7fffffff));
        e = -1;
      }
    }
    const unsigned same = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == (31 - __clz(same))) atomicAdd(&cnt[e], __popc(same));
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const int c = cnt[e];
    if (c) atomicAdd(&hist[e], c);
  }
}

}  // namespace

int moegps_launch_histogram(moegps_ctx* ctx, const int32_t* topk_idx, int32_t* hist, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int64_t R = (int64_t)s.T * s.K;
  MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(hist, 0, sizeof(int32_t) * s.E, st));
  if (R == 0) return MOEGPS_OK;
  int64_t blocks = (R + kHistThreads * 4 - 1) / (kHistThreads * 4);   // ~4 pairs per thread
  if (blocks > 2 * ctx->sm_count) blocks = 2 * ctx->sm_count;
  if (blocks < 1) blocks = 1;
  histogram_kernel<<<(unsigned)blocks, kHistThreads, 0, st>>>(topk_idx, R, s.E, hist, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
