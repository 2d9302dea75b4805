// route: router GEMM fused with bias, warp-shuffle top-K and the gate weights (paper, Section 2).
//
// logits[128 tokens, E] = X_tile * Wr^T on the 5th-generation tensor cores: the token tile is the
// MMA's M (128 rows), the experts its N (E rounded up to 16, at most 256), accumulators in TMEM.
// The kernel is bound by reading X once from HBM, so the grid must cover the chip even when
// T/128 is small: the model dimension is split over the KS CTAs of a thread-block cluster
// (grid = token tiles x KS).  Each CTA streams its slice of X and Wr through a TMA -> shared-memory
// ring into tcgen05.mma, parks its fp32 partial logits in its own shared memory, and after a
// cluster barrier CTA r reduces rows [r*128/KS, (r+1)*128/KS) over all KS partials through
// distributed shared memory in a fixed order (deterministic), adds the bias and lets eight lanes per
// token select the top K by shuffles (route_epilogue.cuh).  When the caller asks for it, the
// per-expert token counts (Eq. 1's n_e) are accumulated on the way: every selection bumps a
// shared-memory counter of its CTA, and each CTA adds its non-zero counters to the global
// histogram once (integer atomics: deterministic).
// Warp roles in the main loop: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = TMEM -> shared-memory drain.  Every mbarrier wait is bounded.
#include "common.cuh"
#include "route_epilogue.cuh"
#include "sm100.cuh"

bool moegps_make_tmap_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols);

namespace {

using namespace sm100;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 384;   // 12 warps: 2 feed the tensor core, 4 drain TMEM, all 12 reduce and select
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
};

// volatile keeps these loads behind the cluster barrier (also a volatile asm) and in program order.
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr));
  return v;
}

// Split-K reduction: CTA `rank` of the cluster owns rows [rank*128/KS, (rank+1)*128/KS) of the tile.
// All threads sum the KS partial logits of those rows in slice order (fixed: deterministic), 16
// bytes per load - consecutive threads read consecutive chunks of a peer's shared memory - and store
// the sums over the CTA's own partials of those rows, which no peer reads.
template <int KS>
__device__ __forceinline__ void reduce_partials(const RouteParams& p, float* partial, uint32_t rank) {
  constexpr int rows_per = BM / KS;
  const int chunks = p.e_pad / 4;
  uint32_t peer[KS];
#pragma unroll
  for (int k = 0; k < KS; ++k) peer[k] = map_to_cta(smem_u32(partial), (uint32_t)k);
  // two chunks per thread and iteration: 2*KS independent 16-byte loads in flight hide the latency of
  // a peer's shared memory
  const int total = rows_per * chunks;
  for (int idx = threadIdx.x; idx < total; idx += 2 * kThreads) {
    const int idx1 = idx + kThreads;
    const bool two = idx1 < total;
    const int word0 = ((int)rank * rows_per + idx / chunks) * p.part_stride + 4 * (idx % chunks);
    const int word1 = two ? ((int)rank * rows_per + idx1 / chunks) * p.part_stride + 4 * (idx1 % chunks) : word0;
    float4 a[KS], b[KS];
#pragma unroll
    for (int k = 0; k < KS; ++k) a[k] = ld_cluster_f32x4(peer[k] + (uint32_t)word0 * 4u);
#pragma unroll
    for (int k = 0; k < KS; ++k) b[k] = ld_cluster_f32x4(peer[k] + (uint32_t)word1 * 4u);
    float4 sa = a[0], sb = b[0];
#pragma unroll
    for (int k = 1; k < KS; ++k) {
      sa.x += a[k].x; sa.y += a[k].y; sa.z += a[k].z; sa.w += a[k].w;
      sb.x += b[k].x; sb.y += b[k].y; sb.z += b[k].z; sb.w += b[k].w;
    }
    *reinterpret_cast<float4*>(partial + word0) = sa;
    if (two) *reinterpret_cast<float4*>(partial + word1) = sb;
  }
}

// Eight lanes per token, four tokens per warp at a time: read the row's logits (already summed
// over the K slices) from shared memory, add the bias, turn the row into order keys (sub-lane l
// holds experts l, l+8, ...) and select.  Every lane of a warp takes part in every shuffle, so rows
// past T (ragged last tile; their logits are zero-filled, finite) are computed like the others and
// only their stores are skipped.
template <int NPL>
__device__ __forceinline__ void select_rows(const RouteParams& p, const float* partial, int row_begin, int rows,
                                            int m0, const float* s_bias, int32_t* __restrict__ topk_idx,
                                            float* __restrict__ topk_w, float* __restrict__ logits_out,
                                            int32_t* cta_hist) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sl = lane & 7, grp = lane >> 3;
  for (int r0 = warp * 4; r0 < rows; r0 += (kThreads / 32) * 4) {     // rows is a multiple of 4
    const int row = row_begin + r0 + grp;
    const int t = m0 + row;
    const bool live = t < p.T;
    const float* prow = partial + (size_t)row * p.part_stride;
    uint32_t key[NPL];
#pragma unroll
    for (int i = 0; i < NPL; ++i) {
      const int e = sl + 8 * i;
      const float v = prow[e < p.E ? e : 0] + s_bias[e < p.E ? e : 0];
      key[i] = e < p.E ? route_order_key(v) : 0u;
      if (logits_out && live && e < p.E) logits_out[(int64_t)t * p.E + e] = v;
    }
    if (topk_idx) {
      const int sel = group8_topk_gate<NPL>(key, p.K, p.gate_mode, live, topk_idx + (int64_t)t * p.K,
                                            topk_w + (int64_t)t * p.K);
      if (cta_hist && live && sel >= 0) atomicAdd(&cta_hist[sel], 1);
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
route_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
             const RouteParams p, const float* __restrict__ bias, int32_t* __restrict__ topk_idx,
             float* __restrict__ topk_w, float* __restrict__ logits_out, int32_t* __restrict__ hist,
             int32_t* __restrict__ status) {
  __shared__ int32_t cta_hist[256];       // this CTA's share of the histogram (used when hist != nullptr)
  __shared__ float s_bias[256];           // fetched before the main loop so that the epilogue does not wait for it
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // [ ring (re-used as the partial-logit buffer) | barriers ]
  const int part_bytes = BM * p.part_stride * 4;
  const int region0 = p.ring_bytes > part_bytes ? p.ring_bytes : part_bytes;
  float* partial = reinterpret_cast<float*>(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + region0);
  uint64_t* full = bars;                 // [stages]
  uint64_t* empty = bars + p.stages;     // [stages]
  uint64_t* acc_full = bars + 2 * p.stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * p.stages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int m0 = blockIdx.x * BM;
  const int nkb = (p.D + BK - 1) / BK;
  const int kb_begin = (int)rank * p.kb_per_cta;
  const int kb_end = min(nkb, kb_begin + p.kb_per_cta);
  const int stage_bytes = kABytes + p.e_pad * 128;

  for (int e = threadIdx.x; e < p.E; e += kThreads) {
    cta_hist[e] = 0;
    s_bias[e] = bias ? bias[e] : 0.f;
  }
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
  } else if (warp < 6) {
    // drain this CTA's partial logits: thread = token row, 32 columns per TMEM load
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    float* prow0 = partial + (size_t)row * p.part_stride;
    if (kb_begin >= kb_end) {
      // an empty K slice (only when D is short): its partial is zero
      for (int c = 0; c < p.e_pad; ++c) prow0[c] = 0.f;
    }
    const bool ok = kb_begin < kb_end && mbar_wait(acc_full, 0, abort_flag);
    tc_fence_after_sync();
    if (ok) {
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
      float* prow = partial + (size_t)row * p.part_stride;
      for (int c0 = 0; c0 < p.e_pad; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(taddr + c0, v);
        tmem_ld_wait();
        // 16-byte stores: with a row stride of 4 (mod 8) words a quarter-warp covers all banks once
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          if (c0 + i < p.e_pad)
            *reinterpret_cast<float4*>(prow + c0 + i) = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]),
                                                                    __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
      }
    }
    tc_fence_before_sync();
  }
  __syncwarp();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    moegps_report(status, MOEGPS_ERR_TIMEOUT, (int)blockIdx.x);
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);    // let copies still in flight land
  }
  __syncwarp();
  cluster_sync_all();           // every CTA's partial is complete and visible cluster-wide

  // reduction + selection: CTA `rank` owns rows [rank*rows_per, (rank+1)*rows_per) of the tile
  switch (p.ks) {
    case 1: break;
    case 2: reduce_partials<2>(p, partial, rank); break;
    case 4: reduce_partials<4>(p, partial, rank); break;
    default: reduce_partials<8>(p, partial, rank); break;
  }
  __syncthreads();
  const int rows_per = BM / p.ks;
  int32_t* const hc = hist ? cta_hist : nullptr;
#define MOEGPS_ROUTE_SELECT(NPL) \
  select_rows<NPL>(p, partial, (int)rank * rows_per, rows_per, m0, s_bias, topk_idx, topk_w, logits_out, hc);
  if (p.E <= 8) { MOEGPS_ROUTE_SELECT(1) }               // experts per lane of an eight-lane group
  else if (p.E <= 16) { MOEGPS_ROUTE_SELECT(2) }
  else if (p.E <= 32) { MOEGPS_ROUTE_SELECT(4) }
  else if (p.E <= 64) { MOEGPS_ROUTE_SELECT(8) }
  else if (p.E <= 128) { MOEGPS_ROUTE_SELECT(16) }
  else { MOEGPS_ROUTE_SELECT(32) }
#undef MOEGPS_ROUTE_SELECT
  __syncwarp();
  cluster_sync_all();           // nobody leaves while a peer may still read its shared memory
  if (hist) {                   // (the barrier above also orders this CTA's shared counters)
    for (int e = threadIdx.x; e < p.E; e += kThreads) {
      const int c = cta_hist[e];
      if (c) atomicAdd(&hist[e], c);
    }
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

}  // namespace

int moegps_launch_route(moegps_ctx* ctx, const void* x, const void* wr, const float* bias, int32_t* topk_idx,
                        float* topk_w, float* logits_out, int32_t* hist, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  if (hist) MOEGPS_CUDA_TRY(ctx, cudaMemsetAsync(hist, 0, sizeof(int32_t) * s.E, st));
  RouteParams p;
  p.T = s.T; p.D = s.D; p.E = s.E; p.K = s.K; p.gate_mode = s.gate_mode;
  p.e_pad = (s.E + 15) / 16 * 16;
  const int stage_bytes = kABytes + p.e_pad * 128;
  p.stages = 196608 / stage_bytes;          // ring of at most 192 KiB
  if (p.stages > 10) p.stages = 10;
  const int nkb = (s.D + BK - 1) / BK;
  const int tiles = (s.T + BM - 1) / BM;
  // split the model dimension until the grid covers most of the chip (cluster size <= 8, a power
  // of two so that 128 rows divide evenly, and every slice keeps at least 4 K blocks)
  int ks = 1;
  while (ks < 8 && tiles * ks * 2 <= ctx->sm_count + ctx->sm_count / 4 && nkb / (ks * 2) >= 4) ks *= 2;
  p.ks = ks;
  p.kb_per_cta = (nkb + ks - 1) / ks;
  if (p.stages > p.kb_per_cta) p.stages = p.kb_per_cta < 2 ? 2 : p.kb_per_cta;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.e_pad) p.tmem_cols *= 2;
  p.ring_bytes = p.stages * stage_bytes;
  p.part_stride = p.e_pad + 4;        // rows 16-byte aligned; 4 (mod 8) words apart: conflict-free 16-byte accesses
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
                                     logits_out, hist, ctx->d_status);
  ctx->launches += 1;
  if (e != cudaSuccess) {
    ctx->last_cuda_error = (int)e;
    return MOEGPS_ERR_CUDA;
  }
  return MOEGPS_OK;
}
