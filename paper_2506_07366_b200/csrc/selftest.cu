// Self-test of the bounded wait every pipelined kernel of this library relies on: a kernel waits on
// an mbarrier that nobody will ever signal, the wait gives up after `limit_cycles` SM cycles, and
// the kernel reports MOEGPS_ERR_TIMEOUT through the status word and returns normally.  Nothing
// faults or hangs, and the context stays usable.
#include "common.cuh"
#include "sm100.cuh"

namespace {

__global__ void bounded_wait_kernel(long long limit_cycles, int32_t* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    abort_flag = 0;
    sm100::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = sm100::mbar_wait(&bar, 0, &abort_flag, 32, limit_cycles);   // phase 0 never completes
    if (!ok) moegps_report(status, MOEGPS_ERR_TIMEOUT, abort_flag);
  }
}

}  // namespace

extern "C" MOEGPS_API int moegps_selftest_bounded_wait(moegps_ctx_t* ctx, int64_t limit_cycles, void* stream) {
  if (!ctx || limit_cycles < 1000 || limit_cycles > 4000000000ll) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  bounded_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}
