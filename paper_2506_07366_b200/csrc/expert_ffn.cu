// expert_ffn: the expert-parallel SwiGLU FFN (paper, Sections 2 and 3.4) over ragged slots, as two
// persistent grouped GEMMs on the 5th-generation tensor cores:
//   GEMM 1:  H  = silu(Xp W1[e]^T) * (Xp W3[e]^T)      (gate and up share the A tile; SwiGLU epilogue)
//   GEMM 2:  Yp = H W2[e]^T
// Tile = 128 rows of one slot x 256 accumulator columns (GEMM 1: 128 gate + 128 up columns).
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (one elected thread; owns TMEM),
// warps 2..9 = epilogue (two per quarter of the 128 TMEM lanes, half the columns each).  A 4-stage ring
// (TMA -> tcgen05.mma) and two TMEM accumulators (mainloop of tile i+1 overlaps the epilogue of tile
// i) are handed around with mbarriers; every wait is bounded and raises an abort flag on expiry.
// Tiles are enumerated on the device from slot_row_off (no host round trip): slot-major, then
// column tile, then row tile, so that CTAs working at the same time share weight tiles in L2.
//
// The launch shape is a template parameter (ring depth, accumulators, epilogue warps, CTAs per SM).
// One shape is in use: 1 CTA per SM, 4-stage ring, two accumulators, 8 epilogue warps.  A shape with
// two smaller CTAs per SM (2-stage rings, one accumulator and 4 epilogue warps each), meant to let a
// weight-streaming tile of a short slot overlap a tensor-bound tile of a long slot on one SM, was
// measured 3-9 % slower on every workload (halving each ring costs more than the overlap returns).
// Also measured and not kept: short slots (at most 128 rows) computed with swapped operands - the two
// 128-row weight tiles of a stage as the MMAs' M, the slot's rows rounded up to 16 as N, transposed
// epilogue - which cuts the tensor time of a 13-row slot eightfold.  Bit-exact, but the many-small-
// expert layer it was meant for gained 2 % (its short slots are bound by streaming their weights,
// not by the padded MMAs) while the bookkeeping cost the other layers 1-2 %.
// And: cutting the tiles of a last round that is at most half full into two 128-column halves (down
// GEMM; 7.35 rounds of tiles on the Mixtral-shaped layer) gained 1 % there and nothing elsewhere, so
// the partial last round is not what separates the down GEMM from the gate+up GEMM.
#include "common.cuh"
#include "sm100.cuh"

namespace {

using namespace sm100;

constexpr int BM = 128;            // rows per tile
constexpr int BNACC = 256;         // accumulator columns per tile
#ifndef MOEGPS_FFN_BK
#define MOEGPS_FFN_BK 64
#endif
// K elements per stage = one swizzle row of BK*2 bytes.  Measured on B200: 64 (128-byte rows, 4
// stages of 48 KiB) beats 32 (64-byte rows, 8 stages of 24 KiB) by about 25 %: TMA moves 128-byte
// rows far more efficiently, which outweighs the deeper ring.
constexpr int BK = MOEGPS_FFN_BK;
constexpr int kRowBytes = BK * 2;
constexpr int kABytes = BM * BK * 2;
constexpr int kBHalfBytes = 128 * BK * 2;
constexpr int kStageBytes = kABytes + 2 * kBHalfBytes;       // 48 KiB
constexpr int kMaxS = 1024;

template <int kStages_, int kAccs_, int kEpiWarps_, int kCtasPerSm_>
struct GemmCfg {
  static constexpr int kStages = kStages_;        // ring depth (48 KiB per stage)
  static constexpr int kAccs = kAccs_;            // 256-column TMEM accumulators
  static constexpr int kEpiWarps = kEpiWarps_;    // 4: one per TMEM lane quarter; 8: two per quarter, half the columns each
  static constexpr int kCtasPerSm = kCtasPerSm_;
  static constexpr int kThreads = 64 + 32 * kEpiWarps_;   // producer warp, MMA warp, epilogue warps
  static constexpr int kTmemCols = 256 * kAccs_;
};
using WideCfg = GemmCfg<256 / BK, 2, 8, 1>;       // 192 KiB of ring

// Per-CTA copy of what decoding a tile needs.  tile_base[s] = first tile index of slot s.
struct __align__(16) Tables {
  int32_t tile_base[kMaxS + 1];
};

constexpr int kStageRowBytes = 80;                 // epilogue staging: 64 payload bytes per row, conflict-free pitch
constexpr int kStagingBytesPerWarp = 32 * kStageRowBytes;

template <class Cfg>
constexpr size_t smem_bytes_of() {
  return 1024 /* alignment slack */ + (size_t)Cfg::kStages * kStageBytes + sizeof(Tables) + 256 +
         (size_t)Cfg::kEpiWarps * kStagingBytesPerWarp;
}
static_assert(smem_bytes_of<WideCfg>() <= 227 * 1024, "one CTA per SM");

struct TileCoord {
  int m0;        // first row of the tile in the permuted buffer
  int row_end;   // one past the last row of the slot's extent
  int n_tile;
  int expert;
};

__device__ __forceinline__ TileCoord decode_tile(const Tables& tb, const int32_t* __restrict__ slot_row_off,
                                               const int32_t* __restrict__ slot_expert, int S, int tile, int n_tiles) {
  int lo = 0, hi = S;                 // find s with tile_base[s] <= tile < tile_base[s+1]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tb.tile_base[mid] <= tile) lo = mid; else hi = mid;
  }
  const int s = lo;
  const int local = tile - tb.tile_base[s];
  const int mt = (tb.tile_base[s + 1] - tb.tile_base[s]) / n_tiles;   // row tiles of this slot
  TileCoord c;
  c.n_tile = local / mt;
  // (the slot tables are a few KiB that every CTA reads: they stay in L1/L2; only slots that passed
  // the checks of the table build own tiles, so these values are in range)
  c.m0 = __ldg(slot_row_off + s) + (local % mt) * BM;
  c.row_end = __ldg(slot_row_off + s + 1);
  c.expert = __ldg(slot_expert + s);
  return c;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// silu(g) = g / (1 + exp(-g)) = g * (0.5 + 0.5 tanh(g / 2)), with the hardware tanh approximation
// (relative error about 2^-11; the product is rounded to bf16, 2^-9, right after).
__device__ __forceinline__ float silu_fast(float g) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
  return g * fmaf(0.5f, t, 0.5f);
}

// Epilogue of one tile for one warp: 32 accumulator rows (one per lane) x half of the tile's output
// columns, TMEM -> registers -> bf16 -> shared-memory staging -> global.
// kSwiGLU: columns [0,128) are the gate and [128,256) the up projection; 128 outputs silu(g)*u.
// [c_begin, c_end) are the output columns this warp drains (with eight epilogue warps two share each
// quarter of the TMEM lanes and take half the columns each).  A lane owns one row, so storing straight from registers would
// scatter 16-byte pieces over 32 rows per instruction - measured to cost the main loop 5-14 % of its
// L2/HBM throughput.  Instead each 32-column chunk (64 bytes per row) goes through a per-warp
// staging buffer (rows 80 bytes apart: conflict-free) and is written out with four lanes per row,
// i.e. whole 64-byte segments.  `row0` is the first of the warp's 32 rows, `row_end` the slot's end.
template <bool kSwiGLU>
__device__ __forceinline__ void drain_tile(uint32_t taddr, uint8_t* staging, int lane, __nv_bfloat16* out,
                                           int row0, int row_end, int col0, int n_dim, int c_begin, int c_end) {
#pragma unroll 1
  for (int c0 = c_begin; c0 < c_end; c0 += 32) {
    uint32_t o[16];
    if constexpr (kSwiGLU) {
      uint32_t g[32], u[32];
      tmem_ld32(taddr + c0, g);
      tmem_ld32(taddr + 128 + c0, u);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
        o[i] = pack_bf16(silu_fast(g0) * __uint_as_float(u[2 * i]), silu_fast(g1) * __uint_as_float(u[2 * i + 1]));
      }
    } else {
      uint32_t a[32];
      tmem_ld32(taddr + c0, a);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i] = pack_bf16(__uint_as_float(a[2 * i]), __uint_as_float(a[2 * i + 1]));
    }
    uint4* mine = reinterpret_cast<uint4*>(staging + lane * kStageRowBytes);
#pragma unroll
    for (int v = 0; v < 4; ++v) mine[v] = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
    __syncwarp();
    const int piece = lane & 3;                       // which 16 bytes of the row's 64
    const int col = col0 + c0 + 8 * piece;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int r = it * 8 + (lane >> 2);
      const uint4 val = *reinterpret_cast<const uint4*>(staging + r * kStageRowBytes + piece * 16);
      const int row = row0 + r;
      if (row < row_end && col + 8 <= n_dim) *reinterpret_cast<uint4*>(out + (size_t)row * n_dim + col) = val;
    }
    __syncwarp();
  }
}

// kSwiGLU = true : out[row, n_tile*128 + c] = silu(acc[c]) * acc[128 + c],  c < 128
// kSwiGLU = false: out[row, n_tile*256 + c] = acc[c],                        c < 256
template <bool kSwiGLU, class Cfg>
__global__ void __launch_bounds__(Cfg::kThreads, Cfg::kCtasPerSm)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                    const __grid_constant__ CUtensorMap tm_b1, const int32_t* __restrict__ slot_row_off,
                    const int32_t* __restrict__ slot_expert, int S, int E, int n_dim, int k_dim, int rcap,
                    __nv_bfloat16* __restrict__ out, int32_t* __restrict__ status) {
  constexpr int kStages = Cfg::kStages, kAccs = Cfg::kAccs, kThreads = Cfg::kThreads;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_mem = smem;                                          // kStages x (A | B0 | B1), 1024-aligned
  Tables& tb = *reinterpret_cast<Tables*>(smem + (size_t)kStages * kStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kStages * kStageBytes + sizeof(Tables));
  uint64_t* full = bars;                  // [kStages]  TMA -> MMA
  uint64_t* empty = bars + kStages;       // [kStages]  MMA -> TMA
  uint64_t* acc_full = bars + 2 * kStages;           // [kAccs]  MMA -> epilogue
  uint64_t* acc_empty = bars + 2 * kStages + kAccs;  // [kAccs]  epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 2 * kAccs);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* warp_tiles = const_cast<int*>(reinterpret_cast<volatile int*>(tmem_slot + 2));   // [32] scan scratch

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cols_per_tile = kSwiGLU ? 128 : 256;
  const int n_tiles = (n_dim + cols_per_tile - 1) / cols_per_tile;
  const int num_kb = (k_dim + BK - 1) / BK;

  // ---------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < kAccs; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], Cfg::kEpiWarps); }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b0);
    prefetch_tensormap(&tm_b1);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, Cfg::kTmemCols);
    tmem_relinquish();
  }
  // tiles per slot.  A slot whose extent is not inside [0, rcap] (offsets negative, decreasing or
  // past the buffers) gets no tiles: nothing is read or written for it, and the caller is told.
  for (int s = threadIdx.x; s <= kMaxS; s += kThreads) {
    int cnt = 0;
    if (s < S) {
      const int lo = slot_row_off[s], hi = slot_row_off[s + 1];
      const int e = slot_expert[s];
      if (lo < 0 || hi < lo || hi > rcap) {
        if (blockIdx.x == 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, s);
      } else if (hi > lo && e >= 0 && e < E) {
        cnt = ((hi - lo + BM - 1) / BM) * n_tiles;
      } else if (hi > lo && e >= E) {
        if (blockIdx.x == 0) moegps_report(status, MOEGPS_ERR_BAD_INDEX, s);
      }
    }
    tb.tile_base[s] = cnt;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // exclusive prefix sum of the counts (warp 0: lane l owns entries 33 l .. 33 l + 32; 32 * 33 > kMaxS)
  if (warp == 0) {
    constexpr int kPer = (kMaxS + 1 + 31) / 32;
    int v[kPer], sum = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int s = lane * kPer + i;
      v[i] = s <= kMaxS ? tb.tile_base[s] : 0;
      sum += v[i];
    }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    int run = incl - sum;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int s = lane * kPer + i;
      if (s <= kMaxS) tb.tile_base[s] = run;
      run += v[i];
    }
    if (lane == 31) warp_tiles[0] = incl;
  }
  __syncthreads();
  const uint32_t tmem_base = *tmem_slot;
  const int total_tiles = warp_tiles[0];

  // ---------------------------------------------------------------- roles
  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        const TileCoord tc = decode_tile(tb, slot_row_off, slot_expert, S, tile, n_tiles);
        const int nb0 = tc.n_tile * cols_per_tile;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* sa = stage_mem + (size_t)stage * kStageBytes;
          mbar_arrive_expect_tx(&full[stage], kStageBytes);
          tma_load_2d(sa, &tm_a, &full[stage], kb * BK, tc.m0);
          tma_load_3d(sa + kABytes, &tm_b0, &full[stage], kb * BK, nb0, tc.expert);
          tma_load_3d(sa + kABytes + kBHalfBytes, &tm_b1, &full[stage], kb * BK, kSwiGLU ? nb0 : nb0 + 128,
                      tc.expert);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let copies that are still in flight land before the CTA retires
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(BM, BNACC);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BNACC;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(stage_mem + (size_t)stage * kStageBytes);
          const uint64_t da = smem_desc_k<kRowBytes>(sa);
          const uint64_t db = smem_desc_k<kRowBytes>(sa + kABytes);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)      // 16 bf16 = 32 bytes per MMA along K
            mma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0);
          mma_commit(&empty[stage]);             // frees the stage when these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        mma_commit(&acc_full[acc]);              // accumulator complete
        if (++acc == kAccs) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
      }
    }
  } else {
    const int quarter = warp & 3;                 // TMEM lanes this warp may read
    constexpr int kOutCols = kSwiGLU ? 128 : 256; // output columns of a tile
    constexpr int kShare = kOutCols / (Cfg::kEpiWarps / 4);          // columns per warp of a lane quarter
    const int c_begin = ((warp - 2) >> 2) * kShare;
    uint8_t* staging = smem + (size_t)kStages * kStageBytes + sizeof(Tables) + 256 + (warp - 2) * kStagingBytesPerWarp;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
      const TileCoord tc = decode_tile(tb, slot_row_off, slot_expert, S, tile, n_tiles);
      if (!mbar_wait(&acc_full[acc], acc_phase, abort_flag, 256)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BNACC;
      const int col0 = tc.n_tile * cols_per_tile;
      drain_tile<kSwiGLU>(taddr, staging, lane, out, tc.m0 + quarter * 32, tc.row_end, col0, n_dim, c_begin,
                          c_begin + kShare);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
      if (++acc == kAccs) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) moegps_report(status, MOEGPS_ERR_TIMEOUT, (int)blockIdx.x);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

namespace {
CUtensorMapSwizzle swizzle_for(uint32_t box_cols) {   // swizzle span = the box's row length in bytes
  return box_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                                      : CU_TENSOR_MAP_SWIZZLE_32B);
}
}  // namespace

// bf16 [rows, cols] row-major; box = box_cols (64, 32 or 16) columns x box_rows rows, swizzle span =
// the box's row length, zero fill outside.
bool moegps_make_tmap_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_cols), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 [batch, rows, cols]; box = box_cols columns x box_rows rows x 1 batch entry.
bool moegps_make_tmap_3d(CUtensorMap* tm, const void* base, uint64_t batch, uint64_t rows, uint64_t cols,
                         uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {cols, rows, batch};
  const cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
  const cuuint32_t box[3] = {box_cols, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(box_cols), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

int tmap_failed(moegps_ctx* ctx) {
  ctx->last_cuda_error = (int)cudaErrorInvalidValue;
  return MOEGPS_ERR_CUDA;
}

template <bool kSwiGLU, class Cfg>
int launch_gemm(moegps_ctx* ctx, bool* attr_done, const CUtensorMap& ta, const CUtensorMap& tb0, const CUtensorMap& tb1,
                const int32_t* slot_row_off, const int32_t* slot_expert, int n_dim, int k_dim, void* out,
                cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  constexpr size_t smem = smem_bytes_of<Cfg>();
  if (!*attr_done) {
    MOEGPS_CUDA_TRY(ctx, cudaFuncSetAttribute(grouped_gemm_kernel<kSwiGLU, Cfg>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    *attr_done = true;
  }
  grouped_gemm_kernel<kSwiGLU, Cfg><<<ctx->sm_count * Cfg::kCtasPerSm, Cfg::kThreads, smem, st>>>(
      ta, tb0, tb1, slot_row_off, slot_expert, s.S, s.E, n_dim, k_dim, (int)moegps_rcap_of(s),
      static_cast<__nv_bfloat16*>(out), ctx->d_status);
  MOEGPS_AFTER_LAUNCH(ctx);
  return MOEGPS_OK;
}

}  // namespace

int moegps_launch_ffn_gate_up(moegps_ctx* ctx, const void* xp, const int32_t* slot_row_off,
                              const int32_t* slot_expert, const void* w_gate, const void* w_up, void* h_ws,
                              cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const uint64_t rcap = (uint64_t)moegps_rcap_of(s);
  if (!(ctx->tm1_valid && ctx->tm_key1[0] == xp && ctx->tm_key1[1] == w_gate && ctx->tm_key1[2] == w_up)) {
    ctx->tm1_valid = false;
    if (!(moegps_make_tmap_2d(&ctx->tm_xp, xp, rcap, s.D, BM, BK) &&
          moegps_make_tmap_3d(&ctx->tm_w1, w_gate, s.E, s.F, s.D, 128, BK) &&
          moegps_make_tmap_3d(&ctx->tm_w3, w_up, s.E, s.F, s.D, 128, BK)))
      return tmap_failed(ctx);
    ctx->tm_key1[0] = xp; ctx->tm_key1[1] = w_gate; ctx->tm_key1[2] = w_up;
    ctx->tm1_valid = true;
  }
  return launch_gemm<true, WideCfg>(ctx, &ctx->ffn_attr_done[0], ctx->tm_xp, ctx->tm_w1, ctx->tm_w3, slot_row_off,
                                    slot_expert, s.F, s.D, h_ws, st);
}

int moegps_launch_ffn_down(moegps_ctx* ctx, const void* h_ws, const int32_t* slot_row_off,
                           const int32_t* slot_expert, const void* w_down, void* yp, cudaStream_t st) {
  const moegps_shape_t& s = ctx->shape;
  const uint64_t rcap = (uint64_t)moegps_rcap_of(s);
  if (!(ctx->tm2_valid && ctx->tm_key2[0] == h_ws && ctx->tm_key2[1] == w_down)) {
    ctx->tm2_valid = false;
    if (!(moegps_make_tmap_2d(&ctx->tm_h, h_ws, rcap, s.F, BM, BK) &&
          moegps_make_tmap_3d(&ctx->tm_w2, w_down, s.E, s.D, s.F, 128, BK)))
      return tmap_failed(ctx);
    ctx->tm_key2[0] = h_ws; ctx->tm_key2[1] = w_down;
    ctx->tm2_valid = true;
  }
  return launch_gemm<false, WideCfg>(ctx, &ctx->ffn_attr_done[1], ctx->tm_h, ctx->tm_w2, ctx->tm_w2, slot_row_off,
                                     slot_expert, s.D, s.F, yp, st);
}
