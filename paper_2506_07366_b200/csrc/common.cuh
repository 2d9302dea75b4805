// Shared host/device declarations of the moegps library (context, status word, launch helpers).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "moegps.h"

// Layout of the device status word: [0] first error code, [1] detail (index / location), [2..3] unused.
struct moegps_ctx {
  moegps_shape_t shape;
  int device;
  int sm_count;
  int32_t* d_status;        // 4 x int32 on the device
  unsigned long long* d_route_acc;   // behind it: 256 64-bit histogram accumulators of the router (all zero between calls)
  int64_t launches;         // kernels launched through this context
  int last_cuda_error;
  // cached TMA descriptors of the expert FFN, keyed by the base pointers they were built for
  const void* tm_key1[3];   // xp, w_gate, w_up
  CUtensorMap tm_xp, tm_w1, tm_w3;
  bool tm1_valid;
  const void* tm_key2[2];   // h_ws, w_down
  CUtensorMap tm_h, tm_w2;
  bool tm2_valid;
  bool ffn_attr_done[2]; // dynamic shared-memory limit raised: gate+up and down instantiations of the GEMM kernel
  // cached TMA descriptors of the router
  const void* rt_key[2];
  CUtensorMap tm_rx, tm_rw;
  bool rt_valid;
  bool route_attr_done;
  bool dispatch_attr_done;
  bool pack_attr_done;
  bool trace;               // MOEGPS_TRACE was set when the context was created: log every launch to stderr
};

// Host-side launch log (off unless the environment asked for it): ordinal, launcher, shape.
inline void moegps_trace_launch(const moegps_ctx* ctx, const char* where) {
  if (!ctx->trace) return;
  const moegps_shape_t& s = ctx->shape;
  fprintf(stderr, "[moegps] launch %lld %s T=%d D=%d F=%d E=%d K=%d S=%d A=%d\n", (long long)ctx->launches, where, s.T, s.D,
          s.F, s.E, s.K, s.S, s.row_align);
}

#define MOEGPS_CUDA_TRY(ctx, expr)                                   \
  do {                                                               \
    cudaError_t _e = (expr);                                         \
    if (_e != cudaSuccess) {                                         \
      (ctx)->last_cuda_error = (int)_e;                              \
      return MOEGPS_ERR_CUDA;                                        \
    }                                                                \
  } while (0)

// Records a launch (and its launch error, if any).
#define MOEGPS_AFTER_LAUNCH(ctx)                                     \
  do {                                                               \
    (ctx)->launches += 1;                                            \
    moegps_trace_launch((ctx), __func__);                            \
    cudaError_t _e = cudaGetLastError();                             \
    if (_e != cudaSuccess) {                                         \
      (ctx)->last_cuda_error = (int)_e;                              \
      return MOEGPS_ERR_CUDA;                                        \
    }                                                                \
  } while (0)

static inline bool moegps_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static inline int64_t moegps_rcap_of(const moegps_shape_t& s) {
  return (int64_t)s.T * s.K + (int64_t)s.S * (s.row_align - 1);
}

// The status word, the cached tensor maps and the kernel attributes of a context belong to its
// device, so that device must be the calling thread's current one; otherwise nothing is launched.
static inline int moegps_check_device(const moegps_ctx* ctx) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOEGPS_ERR_CUDA;
  return dev == ctx->device ? MOEGPS_OK : MOEGPS_ERR_INVALID_ARG;
}

// First error wins; later ones are dropped.
__device__ __forceinline__ void moegps_report(int32_t* status, int code, int detail) {
  if (atomicCAS(&status[0], 0, code) == 0) status[1] = detail;
}

// dispatch: pairs per warp segment of the stable ranking (see dispatch.cu)
constexpr int kSegPairs = 256;

// Per-step launchers (each validates nothing: the C entry points in api.cu do that).
// seg_cnt != nullptr: the router also stores its per-CTA expert counts, [E][CTAs] expert-major.
int moegps_launch_route(moegps_ctx* ctx, const void* x, const void* wr, const float* bias,
                        int32_t* topk_idx, float* topk_w, float* logits_out, int32_t* hist,
                        int32_t* seg_cnt, cudaStream_t st);
// rows of a token tile that one router CTA owns (= 128 / its split of the model dimension)
int moegps_route_rows_per_cta(const moegps_ctx* ctx);
int moegps_launch_dispatch_prepared(moegps_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                                    const int32_t* replicas, const int32_t* slot_off,
                                    int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row, void* xp,
                                    const void* workspace, cudaStream_t st);
int moegps_launch_histogram(moegps_ctx* ctx, const int32_t* topk_idx, int32_t* hist, cudaStream_t st);
int moegps_launch_plan(moegps_ctx* ctx, const int32_t* pred, int32_t* replicas, int32_t* slot_off,
                       int32_t* slot_expert, int32_t* bound, cudaStream_t st);
int moegps_launch_dispatch(moegps_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                           const int32_t* replicas, const int32_t* slot_off, const int32_t* slot_share,
                           int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row, void* xp, void* workspace,
                           cudaStream_t st);
int moegps_launch_ffn_gate_up(moegps_ctx* ctx, const void* xp, const int32_t* slot_row_off,
                              const int32_t* slot_expert, const void* w_gate, const void* w_up, void* h_ws,
                              cudaStream_t st);
int moegps_launch_ffn_down(moegps_ctx* ctx, const void* h_ws, const int32_t* slot_row_off,
                           const int32_t* slot_expert, const void* w_down, void* yp, cudaStream_t st);
int moegps_launch_combine(moegps_ctx* ctx, const void* yp, const int32_t* pair_row, const float* topk_w,
                          void* out, cudaStream_t st);
