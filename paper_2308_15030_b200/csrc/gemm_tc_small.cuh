// Grouped expert-FFN GEMM for SMALL batches (decode: at most 64 (token, expert) pairs per call).
// SwapMoE Section 2: E_i(x) = W_out * act(W_in * x) per Virtual-Expert slot segment.
//
// With a handful of rows per slot the work is pure weight streaming, and the general kernel's
// stages (one 64-column k-block of a 128-row activation tile plus a weight tile) become tiny
// TMA transactions: the k-loop is then bound by the per-transaction cost and by the few bytes in
// flight.  This variant keeps the same roles (TMA producer, single-thread tcgen05.mma issuer,
// TMEM allocator, four epilogue warps, two TMEM accumulators) but
//   - views both operands through 3-D tensor maps (64 columns, rows, k-block index), so ONE
//     TMA instruction brings `kps` consecutive k-blocks of an operand: a stage is
//     kps * (a_rows * 128 + BN * 128) bytes, sized to ~32-48 KB;
//   - loads only the first a_rows (16/32/64) rows of the activation tile; the MMA still reads
//     128 rows, the rest is whatever lies behind in shared memory and only feeds accumulator
//     lanes whose rows are never stored;
//   - takes the stage count at run time (up to 16).
// Every mbarrier wait is bounded as in tc_gemm_kernel.  ReLU / fp32 / scatter epilogues only
// (a SwiGLU layer uses the general kernel for its first GEMM).
#pragma once
#include "gemm_tc.cuh"

namespace swapmoe {

constexpr int kSmMaxStages = 16;
constexpr int kSmSmemBudget = 196 * 1024;

struct TcSmallArgs {
  TcGemmArgs g;          // C, tiles, n_tiles, status, ldc, n_col_tiles, k_blocks, b_rows_per_phys, row_pair, gate, top_k
  int32_t kps;           // k-blocks per stage (k_blocks % kps == 0)
  int32_t n_stages;
  int32_t a_tile_bytes;  // a_rows * 128: one k-block of the activation box
};

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(ptx::smem_u32(dst)), "l"(map), "r"(ptx::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_gemm_small_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const TcSmallArgs sa) {
  const TcGemmArgs& a = sa.g;
  constexpr int kBTile = BN * kTcBK * 2;                    // one k-block of the weight box
  constexpr uint32_t kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;
  constexpr uint32_t kIdesc = make_idesc_bf16(kTcBM, BN);
  const int kps = sa.kps, n_stages = sa.n_stages, a_tile = sa.a_tile_bytes;
  const int stage_a = kps * a_tile, stage_b = kps * kBTile;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // weight stages, activation stages, then 16 KB the 128-row MMA read of the last activation tile may run into
  unsigned char* sB = smem;
  unsigned char* sA = smem + n_stages * stage_b;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + n_stages * (stage_a + stage_b) + kTcBM * kTcBK * 2);
  uint64_t* full = bars;
  uint64_t* empty = bars + kSmMaxStages;
  uint64_t* acc_full = bars + 2 * kSmMaxStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 128); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 2) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_chunks = a.k_blocks / kps;
  // As in tc_gemm_kernel: with `early_b` the producer requests the weight boxes of its first stages before the
  // dependent-launch wait.
  int pre = 0;
  if (warp == 0 && lane == 0 && a.early_b) {
    const int n_rt = __ldcg(a.n_tiles);
    if ((int)blockIdx.x < n_rt * a.n_col_tiles) {
      const int ct = (int)blockIdx.x / n_rt, rt = (int)blockIdx.x - ct * n_rt;
      const int4 rawd = __ldcg(reinterpret_cast<const int4*>(a.tiles + rt));
      const TileDesc td = *reinterpret_cast<const TileDesc*>(&rawd);
      const int brow = td.phys * a.b_rows_per_phys + ct * BN;
      pre = n_chunks < n_stages ? n_chunks : n_stages;
      for (int c = 0; c < pre; ++c) {
        ptx::mbar_expect_tx(&full[c], (uint32_t)(stage_a + stage_b));
        tma_load_3d(sB + c * stage_b, &tmB, &full[c], 0, brow, c * kps);
      }
    }
  }
  pdl_wait();
  pdl_trigger();
  const int n_row_tiles = *a.n_tiles;
  const int total = n_row_tiles * a.n_col_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        const int ct = t / n_row_tiles, rt = t - ct * n_row_tiles;
        const TileDesc td = a.tiles[rt];
        const int brow = td.phys * a.b_rows_per_phys + ct * BN;
        for (int c = 0; c < n_chunks; ++c) {
          const bool early = t == (int)blockIdx.x && c < pre;    // armed and weights requested above
          if (!early) {
            ok = bounded_wait(&empty[stage], phase ^ 1u, abort_flag, a.status, 31);
            if (!ok) break;
            ptx::mbar_expect_tx(&full[stage], (uint32_t)(stage_a + stage_b));
          }
          tma_load_3d(sA + stage * stage_a, &tmA, &full[stage], 0, td.row0, c * kps);
          if (!early) tma_load_3d(sB + stage * stage_b, &tmB, &full[stage], 0, brow, c * kps);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        ok = bounded_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status, 32);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
        for (int c = 0; c < n_chunks; ++c) {
          ok = bounded_wait(&full[stage], phase, abort_flag, a.status, 33);
          if (!ok) break;
          ptx::tc_fence_after();
          for (int kk = 0; kk < kps; ++kk) {
            const uint64_t da = make_kmajor_sw128_desc(ptx::smem_u32(sA + stage * stage_a + kk * a_tile));
            const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(sB + stage * stage_b + kk * kBTile));
#pragma unroll
            for (int k = 0; k < kTcBK / kTcUmmaK; ++k)
              ptx::umma_bf16(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kIdesc,
                             (c > 0 || kk > 0 || k > 0) ? 1u : 0u);
          }
          ptx::umma_commit(&empty[stage]);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(&acc_full[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 4) {
    // -------------------------------------------------------------------- epilogue
    const int q = warp - 4;
    const int r = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
      const int ct = t / n_row_tiles, rt = t - ct * n_row_tiles;
      const TileDesc td = a.tiles[rt];
      // the row's destination and gate value (two dependent global loads) are fetched while the
      // tile's MMAs are still running
      const bool row_ok = r < td.rows;
      size_t crow = (size_t)(td.row0 + r) * a.ldc + (size_t)ct * BN;
      float gate = 1.f;
      if (EPI == kTcEpiScatterBf16 && row_ok) {
        const int p = a.row_pair[td.row0 + r];
        gate = a.gate[p];
        crow = (size_t)(p / a.top_k) * a.ldc + (size_t)ct * BN;
      }
      ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 34);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld32(taddr + (uint32_t)c0, v);
        ptx::tmem_ld_wait();
        if (row_ok) {
          if (EPI == kTcEpiF32) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(a.C) + crow + c0);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                   __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
          } else {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<bf16*>(a.C) + crow + c0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float f[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                f[j] = __uint_as_float(v[8 * i + j]);
                if (EPI == kTcEpiReluBf16) f[j] = fmaxf(f[j], 0.f);
                if (EPI == kTcEpiScatterBf16) f[j] *= gate;
              }
              dst[i] = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]),
                                  pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
            }
          }
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&acc_empty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- host side
inline bool tc_encode_3d(PFN_encodeTiled enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows, uint32_t box_k) {
  const cuuint64_t dims[3] = {(cuuint64_t)kTcBK, rows, cols / kTcBK};
  const cuuint64_t strides[2] = {cols * 2, (cuuint64_t)kTcBK * 2};
  const cuuint32_t box[3] = {(cuuint32_t)kTcBK, box_rows, box_k};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcSmallGeom {
  int bn_index, bn, kps, n_stages, smem_bytes;
};

// Tile width, k-blocks per stage and stage count of one small-batch GEMM.
inline bool tc_small_geometry(int n, int k_blocks, long long row_tiles, int sm_count, int a_tile_bytes,
                              TcSmallGeom* g) {
  g->bn_index = tc_pick_bn(kBn2Options, 4, n, row_tiles, sm_count, a_tile_bytes, 32);
  if (g->bn_index < 0) return false;
  g->bn = kBn2Options[g->bn_index];
  const int per_kb = a_tile_bytes + g->bn * kTcBK * 2;
  g->kps = 1;
  for (int kps = 8; kps > 1; kps >>= 1)
    if (k_blocks % kps == 0 && kps * per_kb <= 48 * 1024) { g->kps = kps; break; }
  const int stage = g->kps * per_kb;
  int ns = (kSmSmemBudget - kTcBM * kTcBK * 2 - 2048) / stage;
  if (ns > kSmMaxStages) ns = kSmMaxStages;
  if (ns > k_blocks / g->kps) ns = k_blocks / g->kps > 1 ? k_blocks / g->kps : 2;
  if (ns < 2) return false;
  g->n_stages = ns;
  g->smem_bytes = ns * stage + kTcBM * kTcBK * 2 + 2048;
  return true;
}

// Tensor maps and geometry of the last small-batch shape served (a decode loop repeats one shape).
struct TcSmallCache {
  bool valid;
  int a_rows, n_tokens;
  TcSmallGeom g1, g2;
  CUtensorMap mA1, mB1, mA2, mB2;
};

typedef void (*TcSmallKernel)(const CUtensorMap, const CUtensorMap, const TcSmallArgs);

template <int EPI>
inline TcSmallKernel tc_small_kernel_for(int bn_index) {
  switch (bn_index) {
    case 0: return tc_gemm_small_kernel<256, EPI>;
    case 1: return tc_gemm_small_kernel<128, EPI>;
    case 2: return tc_gemm_small_kernel<64, EPI>;
    default: return tc_gemm_small_kernel<32, EPI>;
  }
}

inline bool tc_small_set_attrs() {
  bool ok = true;
  for (int i = 0; i < 4; ++i) {
    ok = ok && cudaFuncSetAttribute(tc_small_kernel_for<kTcEpiReluBf16>(i), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kSmSmemBudget) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(tc_small_kernel_for<kTcEpiF32>(i), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kSmSmemBudget) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(tc_small_kernel_for<kTcEpiScatterBf16>(i),
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, kSmSmemBudget) == cudaSuccess;
  }
  return ok;
}

// Both grouped GEMMs of a ReLU layer for a small batch (pairs <= 64).  Same contract as tc_ffn.
inline int32_t tc_ffn_small(TcState& s, TcSmallCache& cache, const swapmoe_config_t& c, const void* xp, void* h,
                            float* y, void* out, int rows_pad, const void* arena_in, const void* arena_out,
                            const TileDesc* tiles, const int32_t* n_tiles, const int32_t* row_pair,
                            const float* mgate, int max_tiles, int n_tokens, int32_t* status, cudaStream_t st,
                            bool pdl, int64_t* launches, bool* combined, cudaEvent_t between = nullptr) {
  if (!s.enabled || !s.arena_bound) return SWAPMOE_ERR_NOT_READY;
  const long long pairs = (long long)n_tokens * c.top_k;
  int a_rows = 16;
  while (a_rows < pairs) a_rows <<= 1;                       // 16, 32 or 64
  const int a_tile = a_rows * kTcBK * 2;
  const long long row_tiles = pairs < c.K ? pairs : c.K;     // one row tile per touched slot
  if (!cache.valid || cache.a_rows != a_rows || cache.n_tokens != n_tokens) {
    const int P = c.K + c.spare_slots;
    if (!tc_small_geometry(c.d_ff, c.d_model / kTcBK, row_tiles, s.sm_count, a_tile, &cache.g1) ||
        !tc_small_geometry(c.d_model, c.d_ff / kTcBK, row_tiles, s.sm_count, a_tile, &cache.g2))
      return SWAPMOE_ERR_UNSUPPORTED;
    if (!tc_encode_3d(s.encode, &cache.mA1, xp, (uint64_t)rows_pad, (uint64_t)c.d_model, a_rows, cache.g1.kps) ||
        !tc_encode_3d(s.encode, &cache.mB1, arena_in, (uint64_t)P * c.d_ff, (uint64_t)c.d_model, cache.g1.bn,
                      cache.g1.kps) ||
        !tc_encode_3d(s.encode, &cache.mA2, h, (uint64_t)rows_pad, (uint64_t)c.d_ff, a_rows, cache.g2.kps) ||
        !tc_encode_3d(s.encode, &cache.mB2, arena_out, (uint64_t)P * c.d_model, (uint64_t)c.d_ff, cache.g2.bn,
                      cache.g2.kps))
      return SWAPMOE_ERR_CUDA;
    cache.a_rows = a_rows;
    cache.n_tokens = n_tokens;
    cache.valid = true;
  }
  const bool scatter = c.top_k == 1;
  TcSmallArgs a1;
  a1.g.C = h; a1.g.tiles = tiles; a1.g.n_tiles = n_tiles; a1.g.status = status; a1.g.ldc = c.d_ff;
  a1.g.n_col_tiles = c.d_ff / cache.g1.bn; a1.g.k_blocks = c.d_model / kTcBK;
  a1.g.b_rows_per_phys = c.d_ff; a1.g.b_rows_gate = 0; a1.g.a_box_bytes = a_tile; a1.g.row_group = 1 << 30;
  a1.g.row_pair = nullptr; a1.g.gate = nullptr; a1.g.top_k = c.top_k; a1.g.early_b = 0;
  a1.kps = cache.g1.kps; a1.n_stages = cache.g1.n_stages; a1.a_tile_bytes = a_tile;
  long long work = (long long)max_tiles * a1.g.n_col_tiles;
  int grid = work > s.sm_count ? s.sm_count : (int)work;
  if (launch_kernel(tc_small_kernel_for<kTcEpiReluBf16>(cache.g1.bn_index), dim3(grid), dim3(kTcThreads),
                    cache.g1.smem_bytes, st, pdl, cache.mA1, cache.mB1, a1) != cudaSuccess)
    return SWAPMOE_ERR_CUDA;
  ++*launches;
  if (between) cudaEventRecord(between, st);

  TcSmallArgs a2;
  a2.g.C = scatter ? out : static_cast<void*>(y);
  a2.g.tiles = tiles; a2.g.n_tiles = n_tiles; a2.g.status = status; a2.g.ldc = c.d_model;
  a2.g.n_col_tiles = c.d_model / cache.g2.bn; a2.g.k_blocks = c.d_ff / kTcBK;
  a2.g.b_rows_per_phys = c.d_model; a2.g.b_rows_gate = 0; a2.g.a_box_bytes = a_tile; a2.g.row_group = 1 << 30;
  a2.g.row_pair = row_pair; a2.g.gate = mgate; a2.g.top_k = c.top_k; a2.g.early_b = 1;
  a2.kps = cache.g2.kps; a2.n_stages = cache.g2.n_stages; a2.a_tile_bytes = a_tile;
  work = (long long)max_tiles * a2.g.n_col_tiles;
  grid = work > s.sm_count ? s.sm_count : (int)work;
  const TcSmallKernel k2 = scatter ? tc_small_kernel_for<kTcEpiScatterBf16>(cache.g2.bn_index)
                                   : tc_small_kernel_for<kTcEpiF32>(cache.g2.bn_index);
  if (launch_kernel(k2, dim3(grid), dim3(kTcThreads), cache.g2.smem_bytes, st, pdl && between == nullptr,
                    cache.mA2, cache.mB2, a2) != cudaSuccess)
    return SWAPMOE_ERR_CUDA;
  ++*launches;
  *combined = scatter;
  return SWAPMOE_OK;
}

}  // namespace swapmoe
