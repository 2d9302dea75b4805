// route: router GEMM fused with bias, top-K selection and the gate weights (paper, Section 2).
//
// logits[128 tokens, E] = X_tile * Wr^T on the 5th-generation tensor cores: the token tile is the
// MMA's M (128 rows), the experts its N (E rounded up to 16, at most 256), accumulators in TMEM.
// The kernel is bound by reading X once from HBM, so the grid must cover the chip even when
// T/128 is small: the model dimension is split over the KS CTAs of a thread-block cluster
// (grid = token tiles x KS).  Each CTA streams its slice of X and Wr through a TMA -> shared-memory
// ring into tcgen05.mma.  The producer starts streaming as soon as the barriers exist; what the
// epilogue needs besides (bias, counters) is fetched while the stream runs.
//
// Split-K reduction by PUSH: CTA r of the cluster owns rows [r*128/KS, (r+1)*128/KS) of the tile.
// The four drain warps read the CTA's fp32 partial logits from TMEM (one thread per token row) and
// store every row straight into its owner's shared memory (st.shared::cluster; remote stores need no
// round trip), at [source slice][row][expert].  One cluster barrier later each owner sums the KS
// partials of its rows from its OWN shared memory in slice order (fixed: deterministic), adds the
// bias and selects.  The partial buffers share the ring's memory, so a first cluster barrier (arrive
// after the CTA's last MMA has completed, wait just before the first push) guarantees that no peer
// still feeds its tensor core from the memory being overwritten; after the second barrier nobody
// touches a peer's shared memory any more, so CTAs leave independently.
//
// Selection: L lanes per token select by shuffles (route_epilogue.cuh), L chosen so that the rows the
// CTA owns occupy all sixteen warps in one pass.  When the caller asks for it, the per-expert token
// counts (Eq. 1's n_e) are accumulated on the way: every selection bumps a shared-memory counter of
// its CTA; each CTA adds its counters to 64-bit accumulators that belong to the context with one
// atomic per expert (the count in the low half, an arrival mark in the high half; integer atomics:
// deterministic); the thread whose atomic returns the last arrival for its expert holds the finished
// count, stores it to the caller's histogram and zeroes the accumulator for the next call - no
// memset, no fence, no second kernel.  In the fused form (moegps_route_prepare) every CTA also stores
// its counters as one column of the count matrix that the dispatch step ranks pairs with, so that
// dispatch is a single launch.
// Warp roles in the main loop: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = drain.  Every mbarrier wait is bounded.
#include "common.cuh"
#include "route_epilogue.cuh"
#include "sm100.cuh"

bool moegps_make_tmap_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols);

namespace {

using namespace sm100;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 512;   // 16 warps: 2 feed the tensor core, 4 drain TMEM, all 16 reduce and select
constexpr int kABytes = BM * BK * 2;      // 16 KiB of X per stage

struct RouteParams {
  int T, D, E, K, gate_mode;
  int e_pad;        // E rounded up to a multiple of 16
  int stages;
  int ks;           // cluster size = number of K slices
  int kb_per_cta;   // 64-wide K blocks per slice
  int tmem_cols;
  int ring_bytes;   // stages * (kABytes + e_pad * 128)
  int part_stride;  // floats per row of the partial-logit buffer (e_pad + 4)
  int lanes;        // lanes per token in the selection (4, 8, 16 or 32; >= K and >= E/32)
};

__device__ __forceinline__ void st_cluster_f32x4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

// L lanes per token, 32/L tokens per warp at a time: read the row's logits (already summed over the
// K slices, bias added) from shared memory, turn them into order keys (sub-lane l holds experts
// l, l+L, ...) and select.  Every lane of a warp takes part in every shuffle, so rows past T (ragged
// last tile; their logits are zero-filled, finite) are computed like the others and only their
// stores are skipped.
template <int L, int NPL>
__device__ __forceinline__ void select_rows(const RouteParams& p, const float* rows_smem, int rows, int t0,
                                            int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                                            int32_t* cta_hist, bool dry) {
  constexpr int kRowsPerWarp = 32 / L;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sl = lane & (L - 1), grp = lane / L;
  for (int r0 = warp * kRowsPerWarp; r0 < rows; r0 += (kThreads / 32) * kRowsPerWarp) {   // rows % 8 == 0
    const int row = r0 + grp;
    const int t = t0 + row;
    const bool live = t < p.T && !dry;
    const float* prow = rows_smem + (size_t)row * p.part_stride;
    uint32_t key[NPL];
#pragma unroll
    for (int i = 0; i < NPL; ++i) {
      const int e = sl + L * i;
      key[i] = e < p.E ? route_order_key(prow[e]) : 0u;
    }
    const int sel = group_topk_gate<L, NPL>(key, p.K, p.gate_mode, live, topk_idx + (int64_t)t * p.K,
                                            topk_w + (int64_t)t * p.K);
    if (cta_hist && live && sel >= 0) atomicAdd(&cta_hist[sel], 1);
  }
}

template <int L>
__device__ __forceinline__ void select_rows_l(const RouteParams& p, const float* rows_smem, int rows, int t0,
                                              int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                                              int32_t* cta_hist, bool dry) {
  const int per_lane = (p.E + L - 1) / L;        // experts per lane, rounded up to a power of two below
#define MOEGPS_SEL(NPL) select_rows<L, NPL>(p, rows_smem, rows, t0, topk_idx, topk_w, cta_hist, dry)
  if (per_lane <= 1) MOEGPS_SEL(1);
  else if (per_lane <= 2) MOEGPS_SEL(2);
  else if (per_lane <= 4) MOEGPS_SEL(4);
  else if (per_lane <= 8) MOEGPS_SEL(8);
  else if (per_lane <= 16) MOEGPS_SEL(16);
  else MOEGPS_SEL(32);                           // the launcher keeps E <= 32 * L
#undef MOEGPS_SEL
}

// Sum of the KS partial logits of the rows this CTA owns, in slice order, plus the bias, 16 bytes per
// access, into slice 0's rows (and to logits_out for the debug entry point).  Not inlined for the
// same reason as select_stage below: idle warps run it once as a dry run (`dry`: nothing is stored)
// while the tile streams, which brings its code into the instruction cache.
__device__ __noinline__ void reduce_stage(const RouteParams& p, float* partial, const float* s_bias, int rows_per,
                                          int t0, float* __restrict__ logits_out, bool dry) {
  const int chunks = p.e_pad / 4;
  const int slice_words = rows_per * p.part_stride;
  // (the dry run is made by warps 6 and up: they start at the first items so that the body is executed)
  for (int idx = dry ? (int)threadIdx.x - 6 * 32 : (int)threadIdx.x; idx < rows_per * chunks; idx += kThreads) {
    const int r = idx / chunks, c = idx - r * chunks;
    const int word = r * p.part_stride + 4 * c;
    float4 s = *reinterpret_cast<const float4*>(partial + word);
    for (int k = 1; k < p.ks; ++k) {
      const float4 q = *reinterpret_cast<const float4*>(partial + (size_t)k * slice_words + word);
      s.x += q.x; s.y += q.y; s.z += q.z; s.w += q.w;
    }
    const int e = 4 * c;         // (bias of padded experts: s_bias is read below 256 only; their keys are never used)
    s.x += s_bias[e]; s.y += s_bias[e + 1]; s.z += s_bias[e + 2]; s.w += s_bias[e + 3];
    if (dry) continue;
    *reinterpret_cast<float4*>(partial + word) = s;
    if (logits_out && t0 + r < p.T) {
      float* lo = logits_out + (int64_t)(t0 + r) * p.E;
      if (e < p.E) lo[e] = s.x;
      if (e + 1 < p.E) lo[e + 1] = s.y;
      if (e + 2 < p.E) lo[e + 2] = s.z;
      if (e + 3 < p.E) lo[e + 3] = s.w;
    }
  }
}

// The selection stage, deliberately NOT inlined: it is called twice from the kernel - first by the
// warps that have nothing to do while the tile streams, as a dry run (`dry`: garbage rows, nothing
// stored, nothing counted) whose only purpose is to pull this code into the SM's instruction cache,
// then by all warps for real.  The kernel runs once per layer, right after GEMMs that have flushed
// every cache, and without the dry run a large share of the selection phase is spent waiting for
// instruction fetches (the profiler's no_instruction stall was the largest single reason).
__device__ __noinline__ void select_stage(const RouteParams& p, const float* rows_smem, int rows, int t0,
                                          int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                                          int32_t* cta_hist, bool dry) {
  switch (p.lanes) {
    case 4: select_rows_l<4>(p, rows_smem, rows, t0, topk_idx, topk_w, cta_hist, dry); break;
    case 8: select_rows_l<8>(p, rows_smem, rows, t0, topk_idx, topk_w, cta_hist, dry); break;
    case 16: select_rows_l<16>(p, rows_smem, rows, t0, topk_idx, topk_w, cta_hist, dry); break;
    default: select_rows_l<32>(p, rows_smem, rows, t0, topk_idx, topk_w, cta_hist, dry); break;
  }
}

__global__ void __launch_bounds__(kThreads, 1)
route_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
             const RouteParams p, const float* __restrict__ bias, int32_t* __restrict__ topk_idx,
             float* __restrict__ topk_w, float* __restrict__ logits_out, int32_t* __restrict__ hist,
             unsigned long long* __restrict__ acc /* context-owned: [256] (arrivals, sum), zero between calls */,
             int32_t* __restrict__ seg_cnt /* [E][CTAs] count matrix of the dispatch step, or nullptr */,
             int32_t* __restrict__ status) {
  __shared__ int32_t cta_hist[256];       // this CTA's share of the histogram (used when hist != nullptr)
  __shared__ float s_bias[256];           // fetched while the stream runs
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // [ ring, later re-used as the partial-logit buffers | barriers ]
  const int part_bytes = BM * p.part_stride * 4;
  const int region0 = p.ring_bytes > part_bytes ? p.ring_bytes : part_bytes;
  float* partial = reinterpret_cast<float*>(smem);       // [source slice][row of mine][part_stride]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + region0);
  uint64_t* full = bars;                 // [stages]
  uint64_t* empty = bars + p.stages;     // [stages]
  uint64_t* acc_full = bars + 2 * p.stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = p.ks > 1 ? cluster_ctarank() : 0u;
  const int m0 = blockIdx.x * BM;
  const int nkb = (p.D + BK - 1) / BK;
  const int kb_begin = (int)rank * p.kb_per_cta;
  const int kb_end = min(nkb, kb_begin + p.kb_per_cta);
  const int stage_bytes = kABytes + p.e_pad * 128;
  const int rows_per = BM / p.ks;

  // set-up: nothing here waits for global memory, so the stream starts within a few hundred cycles
  if (threadIdx.x < 256) cta_hist[threadIdx.x] = 0;
  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&tm_x);
    prefetch_tensormap(&tm_w);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) break;
        uint8_t* sa = smem + (size_t)stage * stage_bytes;
        mbar_arrive_expect_tx(&full[stage], (uint32_t)stage_bytes);
        tma_load_2d(sa, &tm_x, &full[stage], kb * BK, m0);
        tma_load_2d(sa + kABytes, &tm_w, &full[stage], kb * BK, 0);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
    if (p.ks > 1) { cluster_arrive_release(); cluster_wait_acquire(); }   // #1, see the drain warps
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(BM, p.e_pad);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t sa = smem_u32(smem + (size_t)stage * stage_bytes);
        const uint64_t da = smem_desc_k_sw128(sa);
        const uint64_t db = smem_desc_k_sw128(sa + kABytes);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k)
          mma_bf16(tmem_base, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb > kb_begin) || k > 0);
        mma_commit(&empty[stage]);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
      if (ok && kb_begin < kb_end) mma_commit(acc_full);
    }
    __syncwarp();
    if (p.ks > 1) { cluster_arrive_release(); cluster_wait_acquire(); }   // #1
  } else if (warp < 6) {
    // drain: thread = token row of the tile.  The accumulator is complete once acc_full flips; from
    // then on this CTA's ring is no longer read by its tensor core.
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const bool have = kb_begin < kb_end;          // an empty K slice (only when D is short) contributes zeros
    const bool ok = (!have || mbar_wait(acc_full, 0, abort_flag)) && have;
    tc_fence_after_sync();
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    if (p.ks > 1) cluster_arrive_release();       // #1: my tensor core has finished with my ring
    const int owner = row / rows_per, row_local = row - owner * rows_per;
    const uint32_t local = smem_u32(partial + ((size_t)rank * rows_per + row_local) * p.part_stride);
    const uint32_t dst = p.ks > 1 ? map_to_cta(local, (uint32_t)owner) : local;
    uint32_t cur[32];
    if (ok) { tmem_ld32(taddr, cur); tmem_ld_wait(); }
    if (p.ks > 1) cluster_wait_acquire();         // #1: every peer's ring is free as well
    for (int c0 = 0; c0 < p.e_pad; c0 += 32) {
      uint32_t nxt[32];
      const bool more = c0 + 32 < p.e_pad;
      if (more && ok) tmem_ld32(taddr + c0 + 32, nxt);      // overlaps the stores below
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        if (c0 + i < p.e_pad)
          st_cluster_f32x4(dst + (uint32_t)(c0 + i) * 4u, ok ? __uint_as_float(cur[i]) : 0.f,
                           ok ? __uint_as_float(cur[i + 1]) : 0.f, ok ? __uint_as_float(cur[i + 2]) : 0.f,
                           ok ? __uint_as_float(cur[i + 3]) : 0.f);
      }
      if (more) {
        if (ok) tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) cur[i] = nxt[i];
      }
    }
    tc_fence_before_sync();
  } else {
    // idle warps fetch the bias while the stream runs; it is read after the block barrier below
    for (int e = threadIdx.x - 6 * 32; e < p.E; e += kThreads - 6 * 32) s_bias[e] = bias ? bias[e] : 0.f;
    reduce_stage(p, partial, s_bias, rows_per, m0, nullptr, true);                            // both warm the
    if (topk_idx) select_stage(p, partial, rows_per, m0, topk_idx, topk_w, nullptr, true);   // instruction cache
    if (p.ks > 1) { cluster_arrive_release(); cluster_wait_acquire(); }   // #1
  }
  __syncwarp();
  if (p.ks > 1) {
    cluster_arrive_release();     // #2: my pushes are done ...
    cluster_wait_acquire();       //     ... and so are everybody's into my shared memory
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    moegps_report(status, MOEGPS_ERR_TIMEOUT, (int)blockIdx.x);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);    // let copies still in flight land
  }

  // The rows this CTA owns, tile rows [rank*rows_per, (rank+1)*rows_per): sum over the source slices
  // in slice order, add the bias, 16 bytes per access, into slice 0's rows.
  const int t0 = m0 + (int)rank * rows_per;
  if (*abort_flag == 0) {
    reduce_stage(p, partial, s_bias, rows_per, t0, logits_out, false);
    __syncthreads();
    if (topk_idx) select_stage(p, partial, rows_per, t0, topk_idx, topk_w, hist ? cta_hist : nullptr, false);
  }
  __syncthreads();
  if (warp == 1) {                // TMEM is no longer needed; release it before the tail below
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
  if (hist && (int)threadIdx.x < p.E) {
    // One 64-bit atomic per expert and CTA adds this CTA's count (low half) and marks its arrival
    // (high half); the thread whose atomic returns the last arrival holds the finished count.
    const int n_ctas = (int)(gridDim.x * gridDim.y);
    const int sub = (int)blockIdx.x * p.ks + (int)rank;          // this CTA's column of the count matrix
    const int e = (int)threadIdx.x;
    const int c = cta_hist[e];
    if (seg_cnt) seg_cnt[(int64_t)e * n_ctas + sub] = c;
    const unsigned long long old = atomicAdd(&acc[e], (1ull << 32) | (unsigned long long)(uint32_t)c);
    if ((int)(old >> 32) == n_ctas - 1) {
      hist[e] = (int)(uint32_t)old + c;
      acc[e] = 0;                       // zero again for the next call
    }
  }
}

}  // namespace

namespace {
// How the model dimension is split: until the grid covers most of the chip (cluster size <= 8, a
// power of two so that 128 rows divide evenly, and every slice keeps at least 4 K blocks).
int route_split(const moegps_ctx* ctx) {
  const moegps_shape_t& s = ctx->shape;
  const int nkb = (s.D + BK - 1) / BK;
  const int tiles = (s.T + BM - 1) / BM;
  int ks = 1;
  while (ks < 8 && tiles * ks * 2 <= ctx->sm_count + ctx->sm_count / 4 && nkb / (ks * 2) >= 4) ks *= 2;
  return ks;
}
}  // namespace

int moegps_route_rows_per_cta(const moegps_ctx* ctx) { return BM / route_split(ctx); }

int moegps_launch_route(moegps_ctx* ctx, const void* x, const void* wr, const float* bias, int32_t* topk_idx,
                        float* topk_w, float* logits_out, int32_t* hist, int32_t* seg_cnt,
                        cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  RouteParams p;
  p.T = s.T; p.D = s.D; p.E = s.E; p.K = s.K; p.gate_mode = s.gate_mode;
  p.e_pad = (s.E + 15) / 16 * 16;
  const int stage_bytes = kABytes + p.e_pad * 128;
  p.stages = 196608 / stage_bytes;          // ring of at most 192 KiB
  if (p.stages > 10) p.stages = 10;
  const int nkb = (s.D + BK - 1) / BK;
  const int tiles = (s.T + BM - 1) / BM;
  const int ks = route_split(ctx);
  p.ks = ks;
  p.kb_per_cta = (nkb + ks - 1) / ks;
  if (p.stages > p.kb_per_cta) p.stages = p.kb_per_cta < 2 ? 2 : p.kb_per_cta;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.e_pad) p.tmem_cols *= 2;
  p.ring_bytes = p.stages * stage_bytes;
  p.part_stride = p.e_pad + 4;        // rows 16-byte aligned; 4 (mod 8) words apart: conflict-free 16-byte accesses
  // lanes per token in the selection: the CTA's rows fill its threads in one pass where possible;
  // at least K lanes (sub-lane k stores the k-th selection), at most 32 experts per lane
  int lanes = 4;
  while (lanes < 32 && (lanes * 2 * (BM / ks) <= kThreads || lanes < s.K || s.E > 32 * lanes)) lanes *= 2;
  p.lanes = lanes;
  const int part_bytes = BM * p.part_stride * 4;
  const int region0 = p.ring_bytes > part_bytes ? p.ring_bytes : part_bytes;
  const size_t smem_bytes = 1024 + (size_t)region0 + (2 * p.stages + 1) * 8 + 64;

  if (!(ctx->rt_valid && ctx->rt_key[0] == x && ctx->rt_key[1] == wr)) {
    ctx->rt_valid = false;
    if (!(moegps_make_tmap_2d(&ctx->tm_rx, x, (uint64_t)s.T, (uint64_t)s.D, BM, BK) &&
          moegps_make_tmap_2d(&ctx->tm_rw, wr, (uint64_t)s.E, (uint64_t)s.D, (uint32_t)p.e_pad, BK))) {
      ctx->last_cuda_error = (int)cudaErrorInvalidValue;
      return MOEGPS_ERR_CUDA;
    }
    ctx->rt_key[0] = x; ctx->rt_key[1] = wr;
    ctx->rt_valid = true;
  }
  if (!ctx->route_attr_done) {
    MOEGPS_CUDA_TRY(ctx, cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024));
    ctx->route_attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)tiles, (unsigned)ks, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = (unsigned)ks;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, route_kernel, ctx->tm_rx, ctx->tm_rw, p, bias, topk_idx, topk_w,
                                     logits_out, hist, ctx->d_route_acc, seg_cnt, ctx->d_status);
  ctx->launches += 1;
  moegps_trace_launch(ctx, __func__);
  if (e != cudaSuccess) {
    ctx->last_cuda_error = (int)e;
    return MOEGPS_ERR_CUDA;
  }
  return MOEGPS_OK;
}
