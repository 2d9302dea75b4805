// dispatch: the routing shuffle on one device (paper, Section 2; replica choice of Algorithm 1).
//
// The flat pair list is cut into segments of kSegPairs consecutive pairs, one warp per segment.
//   1. segment_count : per-segment, per-expert pair counts -> workspace[seg][e]; row_pair := -1
//   2. scan_offsets  : per expert an exclusive scan of the counts over segments (in place), and the
//                      slot row offsets from hist / replicas / row_align (block scan)
//   3. scatter_index : every warp re-walks its segment in pair order; the stable rank of a pair is
//                      the segment's base plus the number of earlier same-expert pairs in the segment
//                      (warp match + running counters), from which replica, slot and row follow
//   4. copy_rows     : one warp per token reads the token row once (128-bit loads) and writes it to
//                      its K rows of the permuted buffer (128-bit stores)
// Stable by construction, integer only, no atomics on results => bit-exact and deterministic.
#include "common.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kMaxE = 256;
constexpr int kMaxS = 1024;

__global__ void __launch_bounds__(kThreads)
segment_count_kernel(const int32_t* __restrict__ topk_idx, int64_t R, int E, int32_t* __restrict__ seg_cnt,
                     int nseg, int32_t* __restrict__ row_pair, int64_t Rcap, int32_t* __restrict__ status) {
  __shared__ int32_t cnt[kWarpsPerBlock][kMaxE];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // padding rows keep -1: fill everything, occupied rows are overwritten by scatter_index
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < Rcap; i += (int64_t)gridDim.x * blockDim.x)
    row_pair[i] = -1;
  const int seg = blockIdx.x * kWarpsPerBlock + warp;
  if (seg >= nseg) return;
  for (int e = lane; e < E; e += 32) cnt[warp][e] = 0;
  __syncwarp();
  const int64_t p0 = (int64_t)seg * kSegPairs;
  for (int it = 0; it < kSegPairs / 32; ++it) {
    const int64_t p = p0 + it * 32 + lane;
    int e = -1;
    if (p < R) {
      e = topk_idx[p];
      if (e < 0 || e >= E) {
        moegps_report(status, MOEGPS_ERR_BAD_INDEX, (int)(p & 0x7fffffff));
        e = -1;
      }
    }
    const unsigned same = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == (31 - __clz(same))) cnt[warp][e] += __popc(same);   // one leader per expert
    __syncwarp();
  }
  for (int e = lane; e < E; e += 32) seg_cnt[(int64_t)seg * E + e] = cnt[warp][e];
}

// One CTA of 1024 threads.
__global__ void __launch_bounds__(1024)
scan_offsets_kernel(int32_t* __restrict__ seg_cnt, int nseg, int E, int S, int A,
                    const int32_t* __restrict__ hist, const int32_t* __restrict__ replicas,
                    const int32_t* __restrict__ slot_off, int32_t* __restrict__ slot_row_off,
                    int32_t* __restrict__ status) {
  __shared__ int32_t padded[kMaxS];     // rows reserved for each slot (load rounded up to A)
  __shared__ int32_t warp_tot[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int s = tid; s < S; s += blockDim.x) padded[s] = 0;
  __syncthreads();
  // (a) per expert: exclusive scan of its counts over the segments; lanes stride the segments
  for (int e = warp; e < E; e += 32) {
    int running = 0;
    for (int g0 = 0; g0 < nseg; g0 += 32) {
      const int g = g0 + lane;
      const int c = g < nseg ? seg_cnt[(int64_t)g * E + e] : 0;
      int incl = c;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
      }
      if (g < nseg) seg_cnt[(int64_t)g * E + e] = running + incl - c;
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0 && running != hist[e]) moegps_report(status, MOEGPS_ERR_HIST_MISMATCH, e);
  }
  // (b) slot loads: replica rho of expert e takes ranks floor(rho n/r) .. floor((rho+1) n/r) - 1
  if (tid < E) {
    const long long n = hist[tid];
    const int r = replicas[tid];
    const int so = slot_off[tid];
    if (r < 1 || so < 0 || so + r > S || n < 0) {
      moegps_report(status, MOEGPS_ERR_BAD_INDEX, tid);
    } else {
      for (int rho = 0; rho < r; ++rho) {
        const int load = (int)(((rho + 1) * n) / r - (rho * n) / r);
        padded[so + rho] = (load + A - 1) / A * A;
      }
    }
  }
  __syncthreads();
  // slot starts are multiples of A, so the offsets are a plain prefix sum of the padded loads
  const int v = tid < S ? padded[tid] : 0;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int base = 0;
  for (int wv = 0; wv < warp; ++wv) base += warp_tot[wv];
  if (tid < S) slot_row_off[tid + 1] = base + incl;
  if (tid == 0) slot_row_off[0] = 0;
}

__global__ void __launch_bounds__(kThreads)
scatter_index_kernel(const int32_t* __restrict__ topk_idx, int64_t R, int E, int S, int64_t Rcap,
                     const int32_t* __restrict__ seg_base, int nseg, const int32_t* __restrict__ hist,
                     const int32_t* __restrict__ replicas, const int32_t* __restrict__ slot_off,
                     const int32_t* __restrict__ slot_row_off, int32_t* __restrict__ pair_row,
                     int32_t* __restrict__ row_pair, int32_t* __restrict__ status) {
  __shared__ int32_t running[kWarpsPerBlock][kMaxE];
  __shared__ int32_t s_hist[kMaxE], s_rep[kMaxE], s_so[kMaxE];
  __shared__ int32_t s_sro[kMaxS + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    s_hist[e] = hist[e];
    s_rep[e] = replicas[e];
    s_so[e] = slot_off[e];
  }
  for (int s = threadIdx.x; s <= S; s += blockDim.x) s_sro[s] = slot_row_off[s];
  const int seg = blockIdx.x * kWarpsPerBlock + warp;
  if (seg < nseg)
    for (int e = lane; e < E; e += 32) running[warp][e] = seg_base[(int64_t)seg * E + e];
  __syncthreads();
  if (seg >= nseg) return;
  const int64_t p0 = (int64_t)seg * kSegPairs;
  const unsigned lt = (1u << lane) - 1u;
  for (int it = 0; it < kSegPairs / 32; ++it) {
    const int64_t p = p0 + it * 32 + lane;
    int e = -1;
    if (p < R) {
      e = topk_idx[p];
      if (e < 0 || e >= E) e = -1;       // already reported by segment_count
    }
    const unsigned same = __match_any_sync(0xffffffffu, e);
    int rank = 0;
    if (e >= 0) rank = running[warp][e] + __popc(same & lt);
    __syncwarp();
    if (e >= 0 && lane == (31 - __clz(same))) running[warp][e] += __popc(same);
    __syncwarp();
    if (e >= 0) {
      const long long n = s_hist[e];
      const int r = s_rep[e];
      if (n <= 0 || r < 1 || rank >= n) {
        moegps_report(status, MOEGPS_ERR_HIST_MISMATCH, e);
      } else {
        const int rho = (int)((((long long)rank + 1) * r - 1) / n);   // replica whose range holds `rank`
        const int start = (int)(((long long)rho * n) / r);
        const int slot = s_so[e] + rho;
        const long long row = slot <= S - 1 && slot >= 0 ? (long long)s_sro[slot] + (rank - start) : -1;
        if (row < 0 || row >= Rcap) {
          moegps_report(status, MOEGPS_ERR_BAD_INDEX, (int)(p & 0x7fffffff));
        } else {
          pair_row[p] = (int32_t)row;
          row_pair[row] = (int32_t)p;
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads)
copy_rows_kernel(const uint4* __restrict__ x, int T, int K, int chunks /* D*2/16 */,
                 const int32_t* __restrict__ pair_row, int64_t Rcap, uint4* __restrict__ xp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= T) return;
  long long dst[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    int row = j < K ? pair_row[(int64_t)t * K + j] : -1;
    if (row < 0 || row >= Rcap) row = -1;                  // reported by scatter_index; skip here
    dst[j] = row < 0 ? -1 : (long long)row * chunks;
  }
  const uint4* src = x + (int64_t)t * chunks;
  int c = lane;
  for (; c + 96 < chunks; c += 128) {                      // four 16-byte loads in flight per lane
    const uint4 v0 = src[c], v1 = src[c + 32], v2 = src[c + 64], v3 = src[c + 96];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (j < K && dst[j] >= 0) {
        uint4* d = xp + dst[j];
        d[c] = v0; d[c + 32] = v1; d[c + 64] = v2; d[c + 96] = v3;
      }
    }
  }
  for (; c < chunks; c += 32) {
    const uint4 v = src[c];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < K && dst[j] >= 0) xp[dst[j] + c] = v;
  }
}

}  // namespace

int moegps_launch_dispatch(moegps_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                           const int32_t* replicas, const int32_t* slot_off, int32_t* slot_row_off,
                           int32_t* row_pair, int32_t* pair_row, void* xp, void* workspace, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int64_t R = (int64_t)s.T * s.K;
  const int64_t Rcap = moegps_rcap_of(s);
  const int nseg = (int)((R + kSegPairs - 1) / kSegPairs);
  int32_t* seg = static_cast<int32_t*>(workspace);
  int blocks = (nseg + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (blocks < 1) blocks = 1;
  segment_count_kernel<<<blocks, kThreads, 0, st>>>(topk_idx, R, s.E, seg, nseg, row_pair, Rcap, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  scan_offsets_kernel<<<1, 1024, 0, st>>>(seg, nseg, s.E, s.S, s.row_align, hist, replicas, slot_off,
                                          slot_row_off, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  if (R == 0) return MOEGPS_OK;
  scatter_index_kernel<<<blocks, kThreads, 0, st>>>(topk_idx, R, s.E, s.S, Rcap, seg, nseg, hist, replicas,
                                                    slot_off, slot_row_off, pair_row, row_pair, ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  const int tblocks = (s.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  copy_rows_kernel<<<tblocks, kThreads, 0, st>>>(static_cast<const uint4*>(x), s.T, s.K, s.D / 8, pair_row, Rcap,
                                                 static_cast<uint4*>(xp));
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

// ------------------------------------------------------------------------------------------------
// moegps_dispatch_static: dispatch for callers that have no allocator to draw the scratch from.
//
// The per-segment counters live in the fixed device array below instead of a caller-provided
// workspace.  The array is part of the library image: every GPU that loads the library holds its
// 1 MiB until the process exits, whether or not this entry point is ever called.
namespace {

constexpr size_t kStaticScratchInts = 262144;                    // 1 MiB of int32 counters
static __device__ __align__(256) int32_t g_dispatch_scratch[kStaticScratchInts];

constexpr int kMaxDevices = 64;
int32_t* g_scratch_addr[kMaxDevices] = {};                       // device address of the array, per device

}  // namespace

extern "C" MOEGPS_API int moegps_dispatch_static(moegps_ctx_t* ctx, const void* x, const int32_t* topk_idx,
                                                 const int32_t* hist, const int32_t* replicas,
                                                 const int32_t* slot_off, int32_t* slot_row_off,
                                                 int32_t* row_pair, int32_t* pair_row, void* xp, void* stream) {
  if (!ctx) return MOEGPS_ERR_INVALID_ARG;
  const moegps_shape_t& s = ctx->shape;
  const void* always[] = {hist, replicas, slot_off, slot_row_off};
  for (const void* p : always)
    if (!p || !moegps_aligned16(p)) return MOEGPS_ERR_INVALID_ARG;
  if (s.T > 0) {
    const void* with_tokens[] = {x, topk_idx, pair_row, xp};
    for (const void* p : with_tokens)
      if (!p || !moegps_aligned16(p)) return MOEGPS_ERR_INVALID_ARG;
  }
  if (moegps_rcap_of(s) > 0 && (!row_pair || !moegps_aligned16(row_pair))) return MOEGPS_ERR_INVALID_ARG;
  // the scratch holds one int32 per (segment, expert); larger problems must use moegps_dispatch
  const int64_t R = (int64_t)s.T * s.K;
  const int64_t nseg = (R + kSegPairs - 1) / kSegPairs;
  if ((uint64_t)(nseg * s.E) > kStaticScratchInts) return MOEGPS_ERR_STATIC_SCRATCH_EXCEEDED;
  int dev = -1;
  MOEGPS_CUDA_TRY(ctx, cudaGetDevice(&dev));
  if (dev != ctx->device || dev < 0 || dev >= kMaxDevices) return MOEGPS_ERR_INVALID_ARG;
  if (!g_scratch_addr[dev]) {
    // In host code the array's name is only a handle; the address a kernel can use has to be asked
    // for, once per device, with that device current.
    int32_t* p = nullptr;
    MOEGPS_CUDA_TRY(ctx, cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_dispatch_scratch));
    if (!p) return MOEGPS_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  return moegps_launch_dispatch(ctx, x, topk_idx, hist, replicas, slot_off, slot_row_off, row_pair, pair_row, xp,
                                g_scratch_addr[dev], (cudaStream_t)stream);
}
