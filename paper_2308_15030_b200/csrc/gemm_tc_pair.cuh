// Grouped expert GEMM on CTA pairs (SwapMoE Section 2: the experts' FFN restricted to the
// resident slots): two SMs share one 256-row x 256-column tile through tcgen05 `cta_group::2`.
//
// Why a pair: with one SM per 128 x 256 tile every k-block of 64 costs 48 KB of operands (16 KB of
// activations, 32 KB of weights) for 512 tensor-core clocks, which is more than an SM can ingest
// while the tensor pipe runs at full rate.  In a pair each CTA stages its own 128 activation rows
// and HALF of the weight tile (128 of the 256 weight rows); the MMA, issued by the even CTA for
// both, reads the two halves from both shared memories and every CTA's tensor core fills the
// accumulator of its own 128 rows (all 256 columns) in its own TMEM.  That is 32 KB per CTA and
// k-block: the weight bytes an SM pulls are halved, a stage is 32 KB so six stages fit, and the
// accumulator (256 columns) still fits twice, so the epilogue of one tile overlaps the next tile's
// MMAs.
//
// Roles in each CTA (256 threads): warp 0 = TMA producer (own activation rows, own half of the
// weight tile; completion is signalled on the EVEN CTA's `full` barrier, which expects the bytes
// of both CTAs), warp 1 = MMA issuer (even CTA only), warp 2 = TMEM allocation, warps 4-7 =
// epilogue for the CTA's own 128 rows.  `tcgen05.commit` with a two-CTA mask hands the stage back
// to both producers and announces a finished accumulator to both epilogues; the epilogue warps of
// both CTAs arrive on the even CTA's `acc_empty` barrier.  No load uses cluster multicast.  Every
// wait is bounded as in tc_gemm_kernel.
#pragma once
#include "gemm_tc.cuh"

namespace swapmoe {

constexpr int kPairBN = 256;                                  // accumulator columns of the pair's tile
constexpr int kPairHalfRows = kPairBN / 2;                    // weight rows each CTA stages
constexpr int kPairABytes = kTcBM * kTcBK * 2;                // 16 KB
constexpr int kPairBBytes = kPairHalfRows * kTcBK * 2;        // 16 KB
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;
constexpr int kPairStages = (kTcSmemBudget - 2048) / kPairStageBytes;
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + 2048 + kTcEpiStageBytes;

namespace ptx {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tile load whose completion bytes are credited to a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0,
                                                 int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"((unsigned short)3)
      : "memory");
}

}  // namespace ptx

// C tile [256, 256 (128 for SwiGLU)] = epi(A[row0 : row0 + 256, :] * B^T); rows row0 + 128 r .. + 127 belong to
// CTA r of the pair.  `a.tiles` lists 256-row tiles; a tile with <= 128 valid rows leaves the odd CTA without
// activation rows to fetch or results to store (its tensor core multiplies stale shared memory into TMEM columns
// nobody reads).
template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTcThreads, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const TcGemmArgs a) {
  constexpr int kStages = kPairStages;
  constexpr int kOutCols = (EPI == kTcEpiSwigluBf16) ? kPairBN / 2 : kPairBN;
  constexpr uint32_t kTmemCols = 2 * kPairBN;                 // two accumulator sets
  constexpr uint32_t kIdesc = make_idesc_bf16(2 * kTcBM, kPairBN);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* sA = smem;                                   // [stages][128][64] bf16
  unsigned char* sB = smem + kStages * kPairABytes;           // [stages][128][64] bf16
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kPairStageBytes);
  uint64_t* full = bars;                    // [stages]  used in the even CTA
  uint64_t* empty = bars + kStages;         // [stages]  one in each CTA (the commit reaches both)
  uint64_t* acc_full = bars + 2 * kStages;  // [2]       one in each CTA
  uint64_t* acc_empty = acc_full + 2;       // [2]       used in the even CTA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned char* epi_stage = smem + kStages * kPairStageBytes + 1024;   // [4 warps][32 rows][128 bytes]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();               // 0: issues the MMAs
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  constexpr int kTr = (EPI == kTcEpiReluBf16 || EPI == kTcEpiSwigluBf16) ? 2 : 3;   // trace id: GEMM-1 or GEMM-2
  (void)kTr;
  if (threadIdx.x == 0) {
    SWAPMOE_STAMP(kTr, 0);
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 8); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 2) {
    ptx::tmem_alloc_pair(tmem_slot, kTmemCols);               // issued in both CTAs: one allocation for the pair
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();                                    // the peer's barriers are initialised before anyone signals them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // As in tc_gemm_kernel: with `early_b` each producer requests the weight boxes of its first stages before the
  // dependent-launch wait.
  int pre = 0;
  if (warp == 0 && lane == 0 && a.early_b) {
    const int n_rt = __ldcg(a.n_tiles);
    if (pair < n_rt * a.n_col_tiles) {
      int rt, ct;
      decode_tile(pair, n_rt, a.n_col_tiles, a.row_group, &rt, &ct);
      const int4 raw = __ldcg(reinterpret_cast<const int4*>(a.tiles + rt));
      const TileDesc td = *reinterpret_cast<const TileDesc*>(&raw);
      const int brow = td.phys * a.b_rows_per_phys +
                       (EPI == kTcEpiSwigluBf16 ? ct * kPairHalfRows + (int)rank * a.b_rows_gate
                                                : ct * kPairBN + (int)rank * kPairHalfRows);
      pre = a.k_blocks < kStages ? a.k_blocks : kStages;
      for (int kb = 0; kb < pre; ++kb) {
        if (rank == 0)
          ptx::mbar_expect_tx(&full[kb], (uint32_t)((td.rows > kTcBM ? 2 : 1) * kPairABytes + 2 * kPairBBytes));
        ptx::tma_load_2d_pair(sB + kb * kPairBBytes, &tmB, ptx::map_to_cta(ptx::smem_u32(&full[kb]), 0u), kb * kTcBK, brow);
      }
    }
  }
  if (threadIdx.x == 0) SWAPMOE_STAMP(kTr, 1);
  pdl_wait();      // the activations come from the preceding kernel
  pdl_trigger();
  if (threadIdx.x == 0) SWAPMOE_STAMP(kTr, 2);
  const int n_row_tiles = *a.n_tiles;
  const int total = n_row_tiles * a.n_col_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer (both CTAs)
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = pair; t < total && ok; t += n_pairs) {
        int rt, ct;
        decode_tile(t, n_row_tiles, a.n_col_tiles, a.row_group, &rt, &ct);
        const TileDesc td = a.tiles[rt];
        const bool two_halves = td.rows > kTcBM;
        // ReLU / plain: the pair's 256 weight rows are consecutive; SwiGLU: 128 rows of W1 (even CTA) and the
        // same 128 rows of W3 (odd CTA)
        const int brow = td.phys * a.b_rows_per_phys +
                         (EPI == kTcEpiSwigluBf16 ? ct * kPairHalfRows + (int)rank * a.b_rows_gate
                                                  : ct * kPairBN + (int)rank * kPairHalfRows);
        const bool load_a = rank == 0 || two_halves;
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          const bool early = t == pair && kb < pre;          // armed and weights requested above
          if (!early) {
            ok = bounded_wait(&empty[stage], phase ^ 1u, abort_flag, a.status, 11);
            if (!ok) break;
          }
          const uint32_t full_addr = ptx::map_to_cta(ptx::smem_u32(&full[stage]), 0u);
          if (rank == 0 && !early)
            ptx::mbar_expect_tx(&full[stage], (uint32_t)((two_halves ? 2 : 1) * kPairABytes + 2 * kPairBBytes));
          if (load_a)
            ptx::tma_load_2d_pair(sA + stage * kPairABytes, &tmA, full_addr, kb * kTcBK, td.row0 + (int)rank * kTcBM);
          if (!early) ptx::tma_load_2d_pair(sB + stage * kPairBBytes, &tmB, full_addr, kb * kTcBK, brow);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        SWAPMOE_STAMP(kTr, 3);
      }
      if (!ok) {
        // Give copies that are still in flight time to land before shared memory is released.
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ------------------------------------------------------------------ MMA issuer (even CTA, for the pair)
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = pair; t < total && ok; t += n_pairs) {
        ok = bounded_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status, 12);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * kPairBN);
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          ok = bounded_wait(&full[stage], phase, abort_flag, a.status, 13);
          if (!ok) break;
          ptx::tc_fence_after();
          if (t == pair && kb == 0) SWAPMOE_STAMP(kTr, 4);
          const uint64_t da = make_kmajor_sw128_desc(ptx::smem_u32(sA + stage * kPairABytes));
          const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(sB + stage * kPairBBytes));
#pragma unroll
          for (int k = 0; k < kTcBK / kTcUmmaK; ++k)
            ptx::umma_bf16_pair(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kIdesc, (kb > 0 || k > 0) ? 1u : 0u);
          ptx::umma_commit_pair(&empty[stage]);   // frees the stage in both CTAs once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit_pair(&acc_full[acc]);    // accumulator complete, in both CTAs
        SWAPMOE_STAMP(kTr, 5);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 4) {
    // -------------------------------------------------------------------- epilogue (own 128 rows)
    const int q = warp - 4;                    // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;               // row of the CTA's half owned by this thread
    const int rr = (int)rank * kTcBM + r;      // row inside the 256-row tile
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = pair; t < total && ok; t += n_pairs) {
      int rt, ct;
      decode_tile(t, n_row_tiles, a.n_col_tiles, a.row_group, &rt, &ct);
      const TileDesc td = a.tiles[rt];
      const bool row_ok = rr < td.rows;
      // where this thread's row goes (and, for the scatter epilogue, its gate value): two dependent
      // global loads, fetched while the tile's MMAs are still running
      int drow = row_ok ? td.row0 + rr : -1;     // output row of C, -1: not stored
      float gate = 1.f;
      if (EPI == kTcEpiScatterBf16 && row_ok) {
        const int p = a.row_pair[td.row0 + rr];
        gate = a.gate[p];
        drow = p / a.top_k;
      }
      ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 14);
      if (!ok) break;
      ptx::tc_fence_after();
      if (rank == 0 || td.rows > kTcBM) {      // the odd CTA has nothing to read for a tile of <= 128 rows
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kPairBN);
        unsigned char* dst[8];
        epi_row_pointers(dst, drow, lane, a.C, (size_t)a.ldc, (size_t)ct * kOutCols, EPI == kTcEpiF32 ? 4 : 2);
        epi_store_tile<EPI, kOutCols>(taddr, epi_stage + q * kTcEpiWarpStage, lane, gate, dst);
      }
      ptx::tc_fence_before();
      __syncwarp();
      // one arrival per warp, on the even CTA's barrier: 8 arrivals hand the buffer back to the MMA issuer
      if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&acc_empty[acc]), 0u));
      if (r == 0) SWAPMOE_STAMP(kTr, 6);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();       // neither CTA's shared memory, barriers or TMEM go away while the peer may touch them
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

template <int EPI>
inline bool tc_pair_set_smem_attr() {
  return cudaFuncSetAttribute(tc_gemm_pair_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes) ==
         cudaSuccess;
}

// CTA pairs that can be resident at once (0 when the kernels cannot be launched).
inline int tc_pair_init(int sm_count) {
  if (!(tc_pair_set_smem_attr<kTcEpiReluBf16>() && tc_pair_set_smem_attr<kTcEpiSwigluBf16>() &&
        tc_pair_set_smem_attr<kTcEpiF32>() && tc_pair_set_smem_attr<kTcEpiScatterBf16>())) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (sm_count / 2)); cfg.blockDim = dim3(kTcThreads); cfg.dynamicSmemBytes = kPairSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, tc_gemm_pair_kernel<kTcEpiF32>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n < sm_count / 2 ? n : sm_count / 2;
}

// Runs both grouped GEMMs on CTA pairs over the list of 256-row tiles.  With top_k == 1 the second
// GEMM writes gate * y straight into `out` (*combined = true) and no combine kernel is needed.
inline int32_t tc_ffn_pair(TcState& s, int n_pairs, const swapmoe_config_t& c, void* h, float* y, void* out,
                           const TileDesc* tiles, const int32_t* n_tiles, const int32_t* row_pair, const float* mgate,
                           int max_tiles, int n_tokens, int32_t* status, cudaStream_t st, bool pdl, int64_t* launches,
                           bool* combined, cudaEvent_t between = nullptr, bool gemm2_pairs = true,
                           int row_group_forced = 0) {
  if (!s.enabled || !s.arena_bound || n_pairs < 1) return SWAPMOE_ERR_NOT_READY;
  const bool swiglu = c.act == SWAPMOE_ACT_SWIGLU;
  const bool scatter = c.top_k == 1;
  const int out1 = swiglu ? kPairBN / 2 : kPairBN;
  if (c.d_ff % out1 || c.d_model % kPairBN) return SWAPMOE_ERR_UNSUPPORTED;
  const long long pairs = (long long)n_tokens * c.top_k;
  int row_group = 1 << 30;
  if (row_group_forced > 0) row_group = row_group_forced;
  else if (pairs * (long long)c.d_model * 2 > (48ll << 20)) {
    // groups of about 20 MB of token rows (Mixtral shape, 4096 tokens: 8-12 tiles of 256 rows measure 2.58-2.70 ms
    // per forward, 16 tiles 2.68-2.80, 32 tiles 2.86-3.01, 4 tiles 2.68-2.72, 1 tile 3.0)
    row_group = (int)((20ll << 20) / (2ll * kTcBM * c.d_model * 2));
    if (row_group < 4) row_group = 4;
  }
  TcGemmArgs g1;
  g1.C = h; g1.status = status; g1.ldc = c.d_ff;
  g1.tiles = tiles; g1.n_tiles = n_tiles;
  g1.n_col_tiles = c.d_ff / out1;
  g1.k_blocks = c.d_model / kTcBK;
  g1.b_rows_per_phys = swiglu ? 2 * c.d_ff : c.d_ff;
  g1.b_rows_gate = swiglu ? c.d_ff : 0;
  g1.row_pair = nullptr; g1.gate = nullptr; g1.top_k = c.top_k;
  g1.row_group = row_group;
  g1.a_box_bytes = kPairABytes;
  g1.early_b = 0;
  long long work = (long long)max_tiles * g1.n_col_tiles;
  int grid = 2 * (work > n_pairs ? n_pairs : (int)work);
  // weight boxes of 128 rows: kBn1Options[1] for one input matrix, kBn1Options[0] / 2 for SwiGLU's two
  cudaError_t e = s.only == 2 ? cudaSuccess :
      swiglu ? launch_kernel(tc_gemm_pair_kernel<kTcEpiSwigluBf16>, dim3(grid), dim3(kTcThreads), kPairSmemBytes, st, pdl,
                             s.map_xp[0], s.map_win[0], g1)
             : launch_kernel(tc_gemm_pair_kernel<kTcEpiReluBf16>, dim3(grid), dim3(kTcThreads), kPairSmemBytes, st, pdl,
                             s.map_xp[0], s.map_win[1], g1);
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  if (s.only != 2) ++*launches;
  if (between) cudaEventRecord(between, st);
  if (s.only == 1) { *combined = scatter; return SWAPMOE_OK; }

  TcGemmArgs g2;
  g2.C = scatter ? out : static_cast<void*>(y);
  g2.tiles = tiles; g2.n_tiles = n_tiles; g2.status = status; g2.ldc = c.d_model;
  g2.n_col_tiles = c.d_model / kPairBN;
  g2.k_blocks = c.d_ff / kTcBK;
  g2.b_rows_per_phys = c.d_model;
  g2.b_rows_gate = 0;
  g2.row_pair = row_pair; g2.gate = mgate; g2.top_k = c.top_k;
  g2.row_group = row_group;
  g2.a_box_bytes = kPairABytes;
  g2.early_b = 1;
  work = (long long)max_tiles * g2.n_col_tiles;
  grid = 2 * (work > n_pairs ? n_pairs : (int)work);
  const bool pdl2 = pdl && between == nullptr;
  if (!gemm2_pairs) {
    // one CTA per 256-row tile with two row sub-tiles: the same operand bytes per flop as a pair, and a tile whose
    // second half is empty costs half
    g2.a_box_bytes = kTcBM * kTcBK * 2;
    grid = work > s.sm_count ? s.sm_count : (int)work;
    const TcGemmKernel k = scatter ? tc_gemm_kernel<256, kTcEpiScatterBf16, 2> : tc_gemm_kernel<256, kTcEpiF32, 2>;
    if (launch_kernel(k, dim3(grid), dim3(kTcThreads), TcSmem<256, 2>::kBytes, st, pdl2, s.map_h[0], s.map_wout[0], g2) !=
        cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    ++*launches;
    *combined = scatter;
    return SWAPMOE_OK;
  }
  e = scatter ? launch_kernel(tc_gemm_pair_kernel<kTcEpiScatterBf16>, dim3(grid), dim3(kTcThreads), kPairSmemBytes, st, pdl2,
                              s.map_h[0], s.map_wout[1], g2)
              : launch_kernel(tc_gemm_pair_kernel<kTcEpiF32>, dim3(grid), dim3(kTcThreads), kPairSmemBytes, st, pdl2,
                              s.map_h[0], s.map_wout[1], g2);
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  ++*launches;
  *combined = scatter;
  return SWAPMOE_OK;
}

}  // namespace swapmoe
