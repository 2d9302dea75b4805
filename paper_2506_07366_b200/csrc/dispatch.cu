// dispatch: the routing shuffle on one device (paper, Section 2; replica choice of Algorithm 1).
//
// The flat pair list is cut into segments of kSegPairs consecutive pairs.  Two kernels:
//   1. count      : one CTA per segment counts its pairs per expert (warp match + shared counters)
//                   into the workspace and fills row_pair with -1.
//                   Up to kDirectMaxSeg segments (262144 pairs): the counts are stored expert-major,
//                   workspace[e][seg], and CTA 0 also derives the slot row offsets from hist /
//                   replicas / row_align (they do not depend on the counts) with a block scan.
//                   Longer pair lists (count_scan): counts are stored workspace[seg][e] and the CTA
//                   that finishes last (a ticket counter kept in the call's own scratch, right behind
//                   the count matrix and zeroed on the stream before the launch; no waiting) turns
//                   them into per-expert exclusive prefix sums over the segments before it derives
//                   the offsets.
//   2. rank_copy  : one warp per token.  The stable rank of a pair is its segment's base plus the
//                   number of earlier same-expert pairs inside the segment, which the warp counts
//                   from the segment's indices (a 1 KiB read).  The base is read from the scanned
//                   matrix, or (short lists) summed by the warp from the expert's row of counts -
//                   a coalesced read of at most 4 KiB that replaces the serial scan, which was a
//                   chain of dependent global round trips on one SM.  Replica, slot and row follow
//                   in integer arithmetic.  The warp then reads the token row once (128-bit loads)
//                   and writes it to its K rows of the permuted buffer (128-bit stores).
// Stable by construction, integer only, no atomics on results => bit-exact and deterministic.
#include <atomic>

#include "common.cuh"
#include "slot_offsets.cuh"

namespace {

using slot_offsets::share_total;
using slot_offsets::slot_loads_of_expert;

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kMaxE = 256;
constexpr int kMaxS = slot_offsets::kMaxS;
constexpr int kScanThreads = 1024;
constexpr int kScanSmemBytes = 100 * 1024;  // staging of the count matrix; two such CTAs still fit one SM

static_assert(kSegPairs == 256, "the count kernels assign one thread to each pair of a segment");
static_assert(kMaxS <= 4 * kSegPairs, "count_kernel scans four slots per thread");

constexpr int kDirectMaxSeg = 1024;   // up to this many segments rank_copy sums the counts itself

// Short pair lists: counts only, stored expert-major; CTA 0 also builds slot_row_off.
__global__ void __launch_bounds__(kSegPairs)
count_kernel(const int32_t* __restrict__ topk_idx, int64_t R, int E, int S, int A, int32_t* __restrict__ cnt_t,
             int nseg, int32_t* __restrict__ row_pair, int64_t Rcap, const int32_t* __restrict__ hist,
             const int32_t* __restrict__ replicas, const int32_t* __restrict__ slot_off,
             const int32_t* __restrict__ slot_share, int32_t* __restrict__ slot_row_off, int32_t* status) {
  __shared__ int32_t cnt[kMaxE];
  __shared__ int32_t padded[kMaxS];
  __shared__ int32_t warp_tot[kSegPairs / 32];
  const int tid = threadIdx.x, lane = tid & 31;
  const int seg = blockIdx.x;
  // padding rows keep -1: fill everything, occupied rows are overwritten by rank_copy
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + tid; i < Rcap; i += (int64_t)gridDim.x * blockDim.x)
    row_pair[i] = -1;
  for (int e = tid; e < E; e += kSegPairs) cnt[e] = 0;
  __syncthreads();
  {
    const int64_t p = (int64_t)seg * kSegPairs + tid;
    int e = -1;
    if (p < R) {
      e = topk_idx[p];
      if (e < 0 || e >= E) {
        moegps_report(status, MOEGPS_ERR_BAD_INDEX, (int)(p & 0x7fffffff));
        e = -1;
      }
    }
    const unsigned same = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == (31 - __clz(same))) atomicAdd(&cnt[e], __popc(same));   // one add per warp and expert
  }
  __syncthreads();
  if (seg < nseg)
    for (int e = tid; e < E; e += kSegPairs) cnt_t[(int64_t)e * nseg + seg] = cnt[e];
  if (blockIdx.x != 0) return;

  // ---- CTA 0: slot row offsets (independent of the counts) ----
  slot_offsets::build_slot_row_off<kSegPairs>(E, S, A, hist, replicas, slot_off, slot_share, padded, warp_tot,
                                              slot_row_off, status);
}

__global__ void __launch_bounds__(kScanThreads)
count_scan_kernel(const int32_t* __restrict__ topk_idx, int64_t R, int E, int S, int A,
                  int32_t* seg_cnt, int nseg, int32_t* __restrict__ row_pair, int64_t Rcap,
                  const int32_t* __restrict__ hist, const int32_t* __restrict__ replicas,
                  const int32_t* __restrict__ slot_off, const int32_t* __restrict__ slot_share,
                  int32_t* __restrict__ slot_row_off, int e_chunk, int32_t* __restrict__ ticket_ctr, int32_t* status) {
  __shared__ int32_t cnt[kMaxE];
  __shared__ int32_t padded[kMaxS];     // rows reserved for each slot (load rounded up to A)
  __shared__ int32_t warp_tot[32];
  __shared__ int is_last;
  extern __shared__ int32_t scan_mat[];   // [nseg][e_chunk] counts, used by the last CTA only
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = blockIdx.x;
  // padding rows keep -1: fill everything, occupied rows are overwritten by rank_copy
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + tid; i < Rcap; i += (int64_t)gridDim.x * blockDim.x)
    row_pair[i] = -1;
  if (tid < E) cnt[tid] = 0;
  __syncthreads();
  if (tid < kSegPairs) {                      // warps 0..7, whole warps
    const int64_t p = (int64_t)seg * kSegPairs + tid;
    int e = -1;
    if (p < R) {
      e = topk_idx[p];
      if (e < 0 || e >= E) {
        moegps_report(status, MOEGPS_ERR_BAD_INDEX, (int)(p & 0x7fffffff));
        e = -1;
      }
    }
    const unsigned same = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == (31 - __clz(same))) atomicAdd(&cnt[e], __popc(same));   // one add per warp and expert
  }
  __syncthreads();
  if (tid < E && seg < nseg) seg_cnt[(int64_t)seg * E + tid] = cnt[tid];
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(ticket_ctr, 1);
    is_last = ticket == (int)gridDim.x - 1;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  // ---- last CTA only: every segment's counts are now visible ----
  for (int s = tid; s < S; s += blockDim.x) padded[s] = 0;
  __syncthreads();
  // (a) per expert: exclusive scan of its counts over the segments.  The count matrix is pulled
  // into shared memory `e_chunk` expert columns at a time (coalesced), thread e walks its column,
  // and the prefix sums are written back (coalesced).
  for (int e0 = 0; e_chunk > 0 && e0 < E; e0 += e_chunk) {
    const int ec = min(e_chunk, E - e0);
    const int ecp = ec | 1;                     // odd row stride: a column walk hits distinct banks
    // thread layout for the copies: tx walks the expert columns (a power of two >= ec lanes wide),
    // ty the segments - no integer divisions in the loops
    int tpr_log = 0;
    while ((1 << tpr_log) < ec && tpr_log < 8) ++tpr_log;
    const int tx = tid & ((1 << tpr_log) - 1), ty = tid >> tpr_log, rows_per_pass = kScanThreads >> tpr_log;
    for (int g0 = ty; g0 < nseg; g0 += 4 * rows_per_pass) {   // four independent loads in flight per thread
      int val[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int g = g0 + u * rows_per_pass;
        val[u] = (g < nseg && tx < ec) ? __ldcg(&seg_cnt[(int64_t)g * E + e0 + tx]) : 0;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int g = g0 + u * rows_per_pass;
        if (g < nseg && tx < ec) scan_mat[g * ecp + tx] = val[u];
      }
    }
    __syncthreads();
    for (int c = warp; c < ec; c += kScanThreads / 32) {      // one warp per expert column
      int running = 0;
      for (int g0 = 0; g0 < nseg; g0 += 32) {
        const int g = g0 + lane;
        const int v = g < nseg ? scan_mat[g * ecp + c] : 0;
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int o = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += o;
        }
        if (g < nseg) scan_mat[g * ecp + c] = running + incl - v;
        running += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0 && running != hist[e0 + c]) moegps_report(status, MOEGPS_ERR_HIST_MISMATCH, e0 + c);
    }
    __syncthreads();
    for (int g = ty; g < nseg; g += rows_per_pass)
      if (tx < ec) seg_cnt[(int64_t)g * E + e0 + tx] = scan_mat[g * ecp + tx];
    __syncthreads();
  }
  // fallback for pair lists too long for shared memory: a warp per expert, lanes stride the segments
  for (int e = warp; e_chunk == 0 && e < E; e += kScanThreads / 32) {
    int running = 0;
    for (int g0 = 0; g0 < nseg; g0 += 32) {
      const int g = g0 + lane;
      const int c = g < nseg ? __ldcg(&seg_cnt[(int64_t)g * E + e]) : 0;
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
  // (b) slot loads
  if (tid < E) slot_loads_of_expert(tid, S, A, hist, replicas, slot_off, slot_share, padded, status);
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

// Second half of the ranking kernels: lane j < K holds pair j of token t with its stable rank
// (my_rank, -1 if the expert index was out of range).  Replica, slot and row follow in integer
// arithmetic; then the warp reads the token row once (128-bit loads) and writes it to its K rows.
__device__ __forceinline__ void place_and_copy(const uint4* __restrict__ x, int t, int K, int chunks, int S, int64_t Rcap,
                                               int my_e, int my_rank, const int32_t* __restrict__ hist,
                                               const int32_t* __restrict__ replicas,
                                               const int32_t* __restrict__ slot_off,
                                               const int32_t* __restrict__ slot_share,
                                               const int32_t* __restrict__ slot_row_off,
                                               int32_t* __restrict__ pair_row, int32_t* __restrict__ row_pair,
                                               uint4* __restrict__ xp, int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  // ---- replica, slot, row (lane j for pair j) ----
  int row = -1;
  if (lane < K && my_rank >= 0) {
    const long long n = hist[my_e];
    const int r = replicas[my_e];
    if (n <= 0 || r < 1 || my_rank >= n) {
      moegps_report(status, MOEGPS_ERR_HIST_MISMATCH, my_e);
    } else {
      const int so = slot_off[my_e];
      int rho, start;
      const long long tot = (so >= 0 && so + r <= S) ? share_total(slot_share, so, r) : 0;
      if (tot > 0) {                                                   // copies take parts in proportion to their shares
        long long cum = 0;
        int end = 0;
        start = 0;
        for (rho = 0; rho < r - 1; ++rho) {
          cum += slot_share[so + rho];
          end = (int)((n * cum) / tot);
          if (my_rank < end) break;
          start = end;
        }
      } else {
        rho = (int)((((long long)my_rank + 1) * r - 1) / n);           // replica whose range holds the rank
        start = (int)(((long long)rho * n) / r);
      }
      const int slot = so + rho;
      const long long rr = (slot >= 0 && slot < S) ? (long long)slot_row_off[slot] + (my_rank - start) : -1;
      if (rr < 0 || rr >= Rcap) {
        moegps_report(status, MOEGPS_ERR_BAD_INDEX, t);
      } else {
        row = (int)rr;
        pair_row[(int64_t)t * K + lane] = row;
        row_pair[row] = (int32_t)((int64_t)t * K + lane);
      }
    }
  }
  long long dst[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int rj = __shfl_sync(0xffffffffu, row, j);
    dst[j] = (j < K && rj >= 0) ? (long long)rj * chunks : -1;
  }
  // ---- row moves ----
  const uint4* src = x + (int64_t)t * chunks;
  int c = lane;
  for (; c + 96 < chunks; c += 128) {                      // four 16-byte loads in flight per lane
    const uint4 v0 = src[c], v1 = src[c + 32], v2 = src[c + 64], v3 = src[c + 96];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (dst[j] >= 0) {
        uint4* d = xp + dst[j];
        d[c] = v0; d[c + 32] = v1; d[c + 64] = v2; d[c + 96] = v3;
      }
    }
  }
  for (; c < chunks; c += 32) {
    const uint4 vv = src[c];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (dst[j] >= 0) xp[dst[j] + c] = vv;
  }
}

// kDirect: `seg_base` holds the raw counts expert-major ([E][nseg]) and the warp sums the expert's
// row up to its segment itself; otherwise it holds the scanned matrix ([nseg][E]).
template <bool kDirect>
__global__ void __launch_bounds__(kThreads)
rank_copy_kernel(const uint4* __restrict__ x, int T, int K, int chunks /* D*2/16 */,
                 const int32_t* __restrict__ topk_idx, int64_t R, int E, int S, int64_t Rcap,
                 const int32_t* __restrict__ seg_base, int nseg, const int32_t* __restrict__ hist,
                 const int32_t* __restrict__ replicas, const int32_t* __restrict__ slot_off,
                 const int32_t* __restrict__ slot_share, const int32_t* __restrict__ slot_row_off,
                 int32_t* __restrict__ pair_row, int32_t* __restrict__ row_pair, uint4* __restrict__ xp,
                 int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (kDirect && blockIdx.x == 0) {
    // the counts must add up to the histogram the caller passed (the scan path checks the same)
    for (int e = warp; e < E; e += kWarpsPerBlock) {
      int tot = 0;
      for (int g = lane; g < nseg; g += 32) tot += seg_base[(int64_t)e * nseg + g];
      tot = __reduce_add_sync(0xffffffffu, tot);
      if (lane == 0 && tot != hist[e]) moegps_report(status, MOEGPS_ERR_HIST_MISMATCH, e);
    }
  }
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= T) return;
  // ---- ranks of this token's K pairs ----
  int my_rank = -1, my_e = -1, my_base = 0;    // lane j < K ends up holding pair j
  int64_t cur_seg = -1;
  int v[kSegPairs / 32];
  int part[8];                                 // this lane's share of the rank of pair j
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    part[j] = 0;
    if (j < K) {
      const int64_t p = (int64_t)t * K + j;
      const int64_t seg = p / kSegPairs;
      if (seg != cur_seg) {                    // (re)load the segment's indices, 8 per lane
        cur_seg = seg;
#pragma unroll
        for (int i = 0; i < kSegPairs / 32; ++i) {
          const int64_t q = seg * kSegPairs + lane + 32 * i;
          v[i] = q < R ? topk_idx[q] : -1;
        }
      }
      const int e = topk_idx[p];
      const int p_local = (int)(p - seg * kSegPairs);
      int c = 0;
#pragma unroll
      for (int i = 0; i < kSegPairs / 32; ++i) c += (lane + 32 * i < p_local && v[i] == e) ? 1 : 0;
      const bool valid = e >= 0 && e < E;
      if (kDirect && valid) {
        const int32_t* row = seg_base + (int64_t)e * nseg;
        for (int g = lane; g < (int)seg; g += 32) c += row[g];
      }
      part[j] = c;
      if (lane == j) {
        my_e = e;
        if (!kDirect && valid) my_base = seg_base[seg * E + e];
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (j < K) {
      const int rank = __reduce_add_sync(0xffffffffu, part[j]);
      if (lane == j) my_rank = (my_e >= 0 && my_e < E) ? my_base + rank : -1;
    }
  }
  place_and_copy(x, t, K, chunks, S, Rcap, my_e, my_rank, hist, replicas, slot_off, slot_share, slot_row_off, pair_row,
                 row_pair, xp, status);
}

// Dispatch after moegps_route_prepare: the count matrix exists already (one column per router CTA,
// i.e. per `rows_per` consecutive tokens, expert-major), so this single kernel derives the offsets,
// ranks, places and copies.  Every block first rebuilds the slot row offsets in its shared memory from
// the finished histogram and the plan (a few hundred integer operations, cheaper than a launch or a
// grid-wide hand-over; block 0 also stores them for the GEMMs).  Then one warp per token: the stable
// rank of a pair = its expert's counts over the earlier columns (a coalesced read by the warp) + the
// same-expert pairs of the earlier tokens of its own column (the K experts of one token are distinct,
// so its own pairs never count).  The first S blocks also mark the padding rows of one slot each
// with -1.
__global__ void __launch_bounds__(kThreads)
rank_copy_prepared_kernel(const uint4* __restrict__ x, int T, int K, int chunks, const int32_t* __restrict__ topk_idx,
                          int E, int S, int A, int64_t Rcap, const int32_t* __restrict__ seg_cnt, int nsub,
                          int rows_per, const int32_t* __restrict__ hist, const int32_t* __restrict__ replicas,
                          const int32_t* __restrict__ slot_off, int32_t* __restrict__ slot_row_off,
                          int32_t* __restrict__ pair_row, int32_t* __restrict__ row_pair, uint4* __restrict__ xp,
                          int32_t* __restrict__ status) {
  __shared__ int32_t s_row_off[kMaxS + 1];
  __shared__ int32_t s_padded[kMaxS];
  __shared__ int32_t s_warp_tot[kThreads / 32];
  __shared__ int pad_begin, pad_end;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  slot_offsets::build_slot_row_off<kThreads>(E, S, A, hist, replicas, slot_off, nullptr, s_padded, s_warp_tot,
                                             s_row_off, status);
  __syncthreads();
  if (blockIdx.x == 0)
    for (int s = threadIdx.x; s <= S; s += kThreads) slot_row_off[s] = s_row_off[s];
  // ---- padding rows of slots blockIdx.x, blockIdx.x + gridDim.x, ... ----
  for (int b = blockIdx.x; b < S; b += gridDim.x) {
    if (threadIdx.x == 0) { pad_begin = 0; pad_end = 0; }
    __syncthreads();
    const int e = threadIdx.x;                       // blockDim = 256 >= E: the thread of the slot's expert answers
    if (e < E) {
      const int so = slot_off[e], r = replicas[e];
      if (r >= 1 && so <= b && b < so + r) {
        const long long n = hist[e];
        const int rho = b - so;
        const int load = (int)(((long long)(rho + 1) * n) / r - ((long long)rho * n) / r);
        pad_begin = s_row_off[b] + load;
        pad_end = s_row_off[b + 1];
      }
    }
    __syncthreads();
    for (int row = pad_begin + threadIdx.x; row < pad_end; row += kThreads)
      if (row >= 0 && row < Rcap) row_pair[row] = -1;
    __syncthreads();
  }
  // ---- and the rows behind the last slot ----
  for (int64_t row = (int64_t)s_row_off[S] + (int64_t)blockIdx.x * kThreads + threadIdx.x; row < Rcap;
       row += (int64_t)gridDim.x * kThreads)
    if (row >= 0) row_pair[row] = -1;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= T) return;
  // ---- ranks of this token's K pairs (lane j ends up holding pair j) ----
  const int sub = t / rows_per;
  const int64_t q_begin = (int64_t)sub * rows_per * K, q_end = (int64_t)t * K;
  int my_e = -1, my_rank = -1;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (j < K) {
      const int e = topk_idx[(int64_t)t * K + j];
      const bool valid = e >= 0 && e < E;
      int c = 0;
      for (int64_t q = q_begin + lane; q < q_end; q += 32) c += topk_idx[q] == e ? 1 : 0;   // earlier tokens of this column
      if (valid) {                                                                          // earlier columns
        const int32_t* cnt_row = seg_cnt + (int64_t)e * nsub;
        for (int g = lane; g < sub; g += 32) c += cnt_row[g];
      }
      const int rank = __reduce_add_sync(0xffffffffu, c);
      if (lane == j) {
        my_e = e;
        my_rank = valid ? rank : -1;
        if (!valid) moegps_report(status, MOEGPS_ERR_BAD_INDEX, t);
      }
    }
  }
  place_and_copy(x, t, K, chunks, S, Rcap, my_e, my_rank, hist, replicas, slot_off, nullptr, s_row_off, pair_row,
                 row_pair, xp, status);
}

}  // namespace

int moegps_launch_dispatch(moegps_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                           const int32_t* replicas, const int32_t* slot_off, const int32_t* slot_share,
                           int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row, void* xp, void* workspace,
                           cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int64_t R = (int64_t)s.T * s.K;
  const int64_t Rcap = moegps_rcap_of(s);
  const int nseg = (int)((R + kSegPairs - 1) / kSegPairs);
  int32_t* seg = static_cast<int32_t*>(workspace);
  // expert columns of the count matrix that fit the scan's shared-memory staging (0 = none: fallback path)
  int e_chunk = nseg > 0 ? kScanSmemBytes / (nseg * (int)sizeof(int32_t)) - 1 : s.E;   // -1: odd row stride
  if (e_chunk > s.E) e_chunk = s.E;
  if (e_chunk < 0) e_chunk = 0;
  const size_t scan_smem = e_chunk > 0 ? (size_t)(e_chunk | 1) * (nseg > 0 ? nseg : 1) * sizeof(int32_t) : 0;
  if (!ctx->dispatch_attr_done) {
    MOEGPS_CUDA_TRY(ctx, cudaFuncSetAttribute(count_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kScanSmemBytes + 1024));
    ctx->dispatch_attr_done = true;
  }
  const bool direct = nseg <= kDirectMaxSeg;
  if (direct) {
    count_kernel<<<nseg > 0 ? nseg : 1, kSegPairs, 0, st>>>(topk_idx, R, s.E, s.S, s.row_align, seg, nseg, row_pair, Rcap,
                                                            hist, replicas, slot_off, slot_share, slot_row_off,
                                                            ctx->d_status);
  } else {
    int32_t* ticket = seg + (int64_t)nseg * s.E;     // the scratch's last word (see moegps_workspace_bytes)
    MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(ticket, 0, sizeof(int32_t), st));
    count_scan_kernel<<<nseg, kScanThreads, scan_smem, st>>>(topk_idx, R, s.E, s.S, s.row_align, seg, nseg, row_pair,
                                                             Rcap, hist, replicas, slot_off, slot_share, slot_row_off,
                                                             e_chunk, ticket, ctx->d_status);
  }
  MOEGPS_AFTER_LAUNCH(ctx);
  if (R == 0) return MOEGPS_OK;
  const int tblocks = (s.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if (direct) {
    rank_copy_kernel<true><<<tblocks, kThreads, 0, st>>>(
        static_cast<const uint4*>(x), s.T, s.K, s.D / 8, topk_idx, R, s.E, s.S, Rcap, seg, nseg, hist, replicas, slot_off,
        slot_share, slot_row_off, pair_row, row_pair, static_cast<uint4*>(xp), ctx->d_status);
  } else {
    rank_copy_kernel<false><<<tblocks, kThreads, 0, st>>>(
        static_cast<const uint4*>(x), s.T, s.K, s.D / 8, topk_idx, R, s.E, s.S, Rcap, seg, nseg, hist, replicas, slot_off,
        slot_share, slot_row_off, pair_row, row_pair, static_cast<uint4*>(xp), ctx->d_status);
  }
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

int moegps_launch_dispatch_prepared(moegps_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* hist,
                                    const int32_t* replicas, const int32_t* slot_off,
                                    int32_t* slot_row_off, int32_t* row_pair, int32_t* pair_row, void* xp,
                                    const void* workspace, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const int rows_per = moegps_route_rows_per_cta(ctx);
  const int nsub = (s.T + 127) / 128 * (128 / rows_per);
  const int tblocks = (s.T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  rank_copy_prepared_kernel<<<tblocks, kThreads, 0, st>>>(
      static_cast<const uint4*>(x), s.T, s.K, s.D / 8, topk_idx, s.E, s.S, s.row_align, moegps_rcap_of(s),
      static_cast<const int32_t*>(workspace), nsub, rows_per, hist, replicas, slot_off, slot_row_off, pair_row, row_pair,
      static_cast<uint4*>(xp), ctx->d_status);
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
// (+ 64: the word behind the largest count matrix is the scan path's ticket counter)
static __device__ __align__(256) int32_t g_dispatch_scratch[kStaticScratchInts + 64];

constexpr int kMaxDevices = 64;
// device address of the array, per device; atomics because host threads may race to the first call
std::atomic<int32_t*> g_scratch_addr[kMaxDevices];

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
  if (int rc = moegps_check_device(ctx)) return rc;
  const int dev = ctx->device;
  if (dev < 0 || dev >= kMaxDevices) return MOEGPS_ERR_INVALID_ARG;
  int32_t* scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // In host code the array's name is only a handle; the address a kernel can use has to be asked
    // for, once per device, with that device current.  (Two threads racing here both get the same
    // answer, so the second store is harmless.)
    MOEGPS_CUDA_TRY(ctx, cudaGetSymbolAddress(reinterpret_cast<void**>(&scratch), g_dispatch_scratch));
    if (!scratch) return MOEGPS_ERR_CUDA;
    g_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  return moegps_launch_dispatch(ctx, x, topk_idx, hist, replicas, slot_off, nullptr, slot_row_off, row_pair, pair_row,
                                xp, scratch, (cudaStream_t)stream);
}
