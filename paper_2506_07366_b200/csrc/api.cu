// C entry points of libmoegps: context management and host-side argument validation.
// Every step validates its arguments here and launches nothing when they are wrong.
#include <new>

#include <stdlib.h>

#include "common.cuh"

namespace {

int check_shape(const moegps_shape_t* s) {
  if (!s) return MOEGPS_ERR_INVALID_ARG;
  if (s->T < 0 || s->D <= 0 || s->F <= 0 || s->E <= 0 || s->K <= 0 || s->S <= 0) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  if (s->K > s->E || s->K > 8 || s->E > 256 || s->S < s->E || s->S > 1024) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  if ((s->D % 8) != 0 || (s->F % 8) != 0) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  const int a = s->row_align;
  if (a < 1 || a > 256 || (a & (a - 1)) != 0) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  if (s->gate_mode != 0 && s->gate_mode != 1) return MOEGPS_ERR_INVALID_ARG;
  if (s->c_max < 0) return MOEGPS_ERR_INVALID_ARG;
  if (moegps_rcap_of(*s) >= (int64_t)INT32_MAX) return MOEGPS_ERR_UNSUPPORTED_SHAPE;
  return MOEGPS_OK;
}

template <typename... P>
bool all_ok(P... ptrs) {
  const void* a[] = {static_cast<const void*>(ptrs)...};
  for (const void* p : a)
    if (p == nullptr || !moegps_aligned16(p)) return false;
  return true;
}

}  // namespace

extern "C" {

int moegps_create(moegps_ctx_t** out, const moegps_shape_t* shape, int device) {
  if (!out) return MOEGPS_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_shape(shape);
  if (rc != MOEGPS_OK) return rc;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return MOEGPS_ERR_CUDA;
  moegps_ctx* ctx = new (std::nothrow) moegps_ctx();
  if (!ctx) return MOEGPS_ERR_CUDA;
  ctx->shape = *shape;
  ctx->device = device;
  ctx->launches = 0;
  ctx->last_cuda_error = 0;
  ctx->tm1_valid = false;
  ctx->tm2_valid = false;
  for (bool& b : ctx->ffn_attr_done) b = false;
  ctx->rt_valid = false;
  ctx->route_attr_done = false;
  ctx->dispatch_attr_done = false;
  ctx->pack_attr_done = false;
  const char* trace = getenv("MOEGPS_TRACE");
  ctx->trace = trace && trace[0] && trace[0] != '0';
  ctx->d_status = nullptr;
  ctx->d_route_acc = nullptr;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
  constexpr size_t kCtxWords = 4 + 2 * 256;      // status word, router accumulators (64-bit)
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, kCtxWords * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, kCtxWords * sizeof(int32_t));
  ctx->d_route_acc = ctx->d_status ? reinterpret_cast<unsigned long long*>(ctx->d_status + 4) : nullptr;
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    return MOEGPS_ERR_CUDA;
  }
  *out = ctx;
  return MOEGPS_OK;
}

int moegps_destroy(moegps_ctx_t* ctx) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (ctx->d_status) cudaFree(ctx->d_status);
  delete ctx;
  return MOEGPS_OK;
}

int64_t moegps_rcap(const moegps_shape_t* shape) {
  if (check_shape(shape) != MOEGPS_OK) return -1;
  return moegps_rcap_of(*shape);
}

size_t moegps_workspace_bytes(const moegps_shape_t* shape) {
  if (check_shape(shape) != MOEGPS_OK) return 0;
  const int64_t R = (int64_t)shape->T * shape->K;
  const int64_t nseg = (R + kSegPairs - 1) / kSegPairs;
  // the per-(segment, expert) count matrix + one word for the scan path's ticket counter; or, for
  // the fused form (moegps_route_prepare), one column per router CTA: the router runs one CTA per
  // 128-token tile, or splits the tiles over up to 8 CTAs while the grid stays within about 1.25x
  // the SM count (bounded here by 320 CTAs)
  const int64_t tiles = ((int64_t)shape->T + 127) / 128;
  const int64_t cols = nseg > (tiles > 320 ? tiles : 320) ? nseg : (tiles > 320 ? tiles : 320);
  size_t bytes = ((size_t)cols * shape->E + 1) * sizeof(int32_t);
  return (bytes + 255) & ~(size_t)255;
}

int moegps_route(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                 int32_t* topk_idx, float* topk_w, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;          // nothing to route (empty tensors have no address)
  if (!all_ok(x, w_router, topk_idx, topk_w)) return MOEGPS_ERR_INVALID_ARG;
  if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_route(ctx, x, w_router, bias, topk_idx, topk_w, nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

int moegps_route_histogram(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                           int32_t* topk_idx, float* topk_w, int32_t* hist, void* stream) {
  if (!ctx || !all_ok(hist)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0)                            // no tokens: the histogram is all zero
    return cudaMemsetAsync(hist, 0, sizeof(int32_t) * ctx->shape.E, (cudaStream_t)stream) == cudaSuccess
               ? MOEGPS_OK : MOEGPS_ERR_CUDA;
  if (!all_ok(x, w_router, topk_idx, topk_w)) return MOEGPS_ERR_INVALID_ARG;
  if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_route(ctx, x, w_router, bias, topk_idx, topk_w, nullptr, hist, nullptr, (cudaStream_t)stream);
}

int moegps_route_prepare(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                         int32_t* topk_idx, float* topk_w, int32_t* hist, void* workspace, void* stream) {
  if (!ctx || !all_ok(hist, workspace)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (ctx->shape.T == 0) {                          // no tokens: the histogram is all zero
    MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(hist, 0, sizeof(int32_t) * ctx->shape.E, st));
    return MOEGPS_OK;
  }
  if (!all_ok(x, w_router, topk_idx, topk_w)) return MOEGPS_ERR_INVALID_ARG;
  if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_route(ctx, x, w_router, bias, topk_idx, topk_w, nullptr, hist, static_cast<int32_t*>(workspace),
                             st);
}

int moegps_dispatch_prepared(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                             const int32_t* replicas, const int32_t* slot_off, int32_t* slot_row_off,
                             int32_t* row_pair, int32_t* pair_row, void* xp, const void* workspace, void* stream) {
  if (!ctx || !all_ok(hist, replicas, slot_off, slot_row_off, workspace)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) {                          // nothing routed: every slot is empty, no padding exists
    MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(slot_row_off, 0, sizeof(int32_t) * (ctx->shape.S + 1), (cudaStream_t)stream));
    return MOEGPS_OK;
  }
  if (!all_ok(x, topk_idx, pair_row, xp, row_pair)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_dispatch_prepared(ctx, x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row,
                                         xp, workspace, (cudaStream_t)stream);
}

int moegps_route_logits(moegps_ctx_t* ctx, const void* x, const void* w_router, const float* bias,
                        float* logits, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;
  if (!all_ok(x, w_router, logits)) return MOEGPS_ERR_INVALID_ARG;
  if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_route(ctx, x, w_router, bias, nullptr, nullptr, logits, nullptr, nullptr, (cudaStream_t)stream);
}

int moegps_histogram(moegps_ctx_t* ctx, const int32_t* topk_idx, int32_t* hist, void* stream) {
  if (!ctx || !all_ok(hist)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T > 0 && !all_ok(topk_idx)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_histogram(ctx, topk_idx, hist, (cudaStream_t)stream);
}

int moegps_plan(moegps_ctx_t* ctx, const int32_t* predicted_hist, int32_t n_slots, int32_t* replicas,
                int32_t* slot_off, int32_t* slot_expert, int32_t* bound, void* stream) {
  if (!ctx || !all_ok(predicted_hist, replicas, slot_off, slot_expert) || !bound) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (reinterpret_cast<uintptr_t>(bound) & 3u) return MOEGPS_ERR_INVALID_ARG;
  if (n_slots != ctx->shape.S) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_plan(ctx, predicted_hist, replicas, slot_off, slot_expert, bound, (cudaStream_t)stream);
}

int moegps_dispatch(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                    const int32_t* replicas, const int32_t* slot_off, int32_t* slot_row_off,
                    int32_t* row_pair, int32_t* pair_row, void* xp, void* workspace, void* stream) {
  if (!ctx || !all_ok(hist, replicas, slot_off, slot_row_off, workspace)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T > 0 && !all_ok(x, topk_idx, pair_row, xp)) return MOEGPS_ERR_INVALID_ARG;
  if (moegps_rcap_of(ctx->shape) > 0 && !all_ok(row_pair)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_dispatch(ctx, x, topk_idx, hist, replicas, slot_off, nullptr, slot_row_off, row_pair, pair_row,
                                xp, workspace, (cudaStream_t)stream);
}

int moegps_dispatch_shares(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                           const int32_t* replicas, const int32_t* slot_off, const int32_t* slot_share,
                           int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row, void* xp, void* workspace,
                           void* stream) {
  if (!ctx || !all_ok(hist, replicas, slot_off, slot_share, slot_row_off, workspace)) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T > 0 && !all_ok(x, topk_idx, pair_row, xp)) return MOEGPS_ERR_INVALID_ARG;
  if (moegps_rcap_of(ctx->shape) > 0 && !all_ok(row_pair)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_dispatch(ctx, x, topk_idx, hist, replicas, slot_off, slot_share, slot_row_off, row_pair,
                                pair_row, xp, workspace, (cudaStream_t)stream);
}

int moegps_expert_ffn(moegps_ctx_t* ctx, const void* xp, const int32_t* slot_row_off,
                      const int32_t* slot_expert, const void* w_gate, const void* w_up, const void* w_down,
                      void* h_ws, void* yp, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;
  if (!all_ok(xp, slot_row_off, slot_expert, w_gate, w_up, w_down, h_ws, yp)) return MOEGPS_ERR_INVALID_ARG;
  int rc = moegps_launch_ffn_gate_up(ctx, xp, slot_row_off, slot_expert, w_gate, w_up, h_ws, (cudaStream_t)stream);
  if (rc != MOEGPS_OK) return rc;
  return moegps_launch_ffn_down(ctx, h_ws, slot_row_off, slot_expert, w_down, yp, (cudaStream_t)stream);
}

int moegps_expert_ffn_gate_up(moegps_ctx_t* ctx, const void* xp, const int32_t* slot_row_off,
                              const int32_t* slot_expert, const void* w_gate, const void* w_up, void* h_ws,
                              void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;
  if (!all_ok(xp, slot_row_off, slot_expert, w_gate, w_up, h_ws)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_ffn_gate_up(ctx, xp, slot_row_off, slot_expert, w_gate, w_up, h_ws, (cudaStream_t)stream);
}

int moegps_expert_ffn_down(moegps_ctx_t* ctx, const void* h_ws, const int32_t* slot_row_off,
                           const int32_t* slot_expert, const void* w_down, void* yp, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;
  if (!all_ok(h_ws, slot_row_off, slot_expert, w_down, yp)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_ffn_down(ctx, h_ws, slot_row_off, slot_expert, w_down, yp, (cudaStream_t)stream);
}

int moegps_combine(moegps_ctx_t* ctx, const void* yp, const int32_t* pair_row, const float* topk_w,
                   void* out, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  if (ctx->shape.T == 0) return MOEGPS_OK;
  if (!all_ok(yp, pair_row, topk_w, out)) return MOEGPS_ERR_INVALID_ARG;
  return moegps_launch_combine(ctx, yp, pair_row, topk_w, out, (cudaStream_t)stream);
}

int moegps_status(moegps_ctx_t* ctx, void* stream, int32_t* host_status) {
  if (!ctx || !host_status) return MOEGPS_ERR_INVALID_ARG;
  if (int rc = moegps_check_device(ctx)) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t h[2] = {0, 0};      // error code and its detail
  MOEGPS_CUDA_TRY(ctx, cudaMemcpyAsync(h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st));
  MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(h), st));
  MOEGPS_CUDA_TRY(ctx, cudaStreamSynchronize(st));
  host_status[0] = h[0];
  return MOEGPS_OK;
}

int64_t moegps_launch_count(const moegps_ctx_t* ctx) { return ctx ? ctx->launches : -1; }

int moegps_last_cuda_error(const moegps_ctx_t* ctx) { return ctx ? ctx->last_cuda_error : 0; }

const char* moegps_error_string(int code) {
  switch (code) {
    case MOEGPS_OK: return "ok";
    case MOEGPS_ERR_INVALID_ARG: return "invalid argument (null/misaligned pointer, n_slots != S, bad mode)";
    case MOEGPS_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case MOEGPS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MOEGPS_ERR_CUDA: return "CUDA call failed";
    case MOEGPS_ERR_UNIMPLEMENTED: return "not implemented";
    case MOEGPS_ERR_BAD_INDEX: return "device saw an index out of range (access skipped)";
    case MOEGPS_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case MOEGPS_ERR_HIST_MISMATCH: return "hist passed to dispatch disagrees with topk_idx";
    case MOEGPS_ERR_STATIC_SCRATCH_EXCEEDED:
      return "problem too large for the built-in scratch of moegps_dispatch_static (ceil(T*K/256)*E > 262144): "
             "use moegps_dispatch with a caller-provided workspace";
    default: return "unknown moegps error";
  }
}

}  // extern "C"
