// Launch logic of the two grouped GEMMs of a bf16 layer on one CTA per tile (tc_gemm_kernel).
// SwapMoE Section 2: E_i(x) per slot.
#pragma once
#include "gemm_tc_pair.cuh"

namespace swapmoe {

// How tc_ffn launches GEMM-1 for a forward of n_tokens.
struct TcGemm1Plan {
  int i1, bn1, out1;        // index into kBn1Options, tile width, output columns per tile
  int n_col_tiles, grid, row_group, ia, a_box_bytes, stages;
  long long row_tiles_est;
};
inline bool tc_plan_gemm1(const TcState& s, const swapmoe_config_t& c, int n_tokens, int mt, int max_tiles,
                          int row_group_forced, TcGemm1Plan* p) {
  const bool swiglu = c.act == SWAPMOE_ACT_SWIGLU;
  // row tiles expected: every touched slot (at most min(pairs, K)) has at least one, and large slots
  // have pairs / 128 in total plus on average half a ragged tile each
  const long long pairs = (long long)n_tokens * c.top_k;
  const long long touched = pairs < c.K ? pairs : c.K;
  const long long by_rows = pairs / kTcBM + touched / 2;
  p->row_tiles_est = touched > by_rows ? touched : by_rows;
  // no tile holds more rows than there are pairs: small batches fetch only the rows that can be valid
  int ia = 0;
  while (ia < 3 && (kTcBM >> (ia + 1)) >= pairs) ++ia;
  if (mt == 2) ia = 0;
  p->ia = ia;
  p->a_box_bytes = (kTcBM >> ia) * kTcBK * 2;
  // Large activation matrices (tens of MB) are walked in groups of 32 row tiles so that a group's
  // rows stay in L2 across its column tiles; small ones are a single group.
  p->row_group = 1 << 30;
  if (row_group_forced > 0) p->row_group = row_group_forced;
  else if (pairs * (long long)c.d_model * 2 > (48ll << 20)) p->row_group = 32;
  p->i1 = tc_pick_bn(kBn1Options, 3, c.d_ff, p->row_tiles_est * mt, s.sm_count, p->a_box_bytes, swiglu ? 64 : 32);
  if (p->i1 < 0) return false;
  p->bn1 = kBn1Options[p->i1];
  p->out1 = swiglu ? p->bn1 / 2 : p->bn1;
  p->n_col_tiles = c.d_ff / p->out1;
  const long long work = (long long)max_tiles * mt * p->n_col_tiles;
  p->grid = work > s.sm_count ? s.sm_count : (int)work;
  p->stages = (kTcSmemBudget - 2048) / (kTcBM * kTcBK * 2 + p->bn1 * kTcBK * 2);
  return true;
}

// Runs both grouped GEMMs.  With top_k == 1 the second GEMM writes gate * y straight into
// `out` (*combined = true) and no combine kernel is needed.
inline int32_t tc_ffn(TcState& s, const swapmoe_config_t& c, void* h, float* y, void* out, const TileDesc* tiles,
                      const int32_t* n_tiles, const TileDesc* tiles128, const int32_t* n_tiles128,
                      const int32_t* row_pair, const float* mgate, int max_tiles, int mt,
                      int n_tokens, int32_t* status, cudaStream_t st, bool pdl, int64_t* launches, bool* combined,
                      cudaEvent_t between = nullptr, int row_group_forced = 0) {
  if (!s.enabled || !s.arena_bound) return SWAPMOE_ERR_NOT_READY;
  const bool swiglu = c.act == SWAPMOE_ACT_SWIGLU;
  const bool scatter = c.top_k == 1;
  // ---- GEMM-1: h = act(xp * W_in^T).  Its k-loop is short (d_model / 64 blocks), so its epilogue must
  // overlap the next tile's MMAs: always one sub-tile per CTA with two TMEM buffers.
  TcGemm1Plan plan;
  if (!tc_plan_gemm1(s, c, n_tokens, mt, max_tiles, row_group_forced, &plan)) return SWAPMOE_ERR_UNSUPPORTED;
  const long long row_tiles_est = plan.row_tiles_est;
  const int ia = plan.ia, a_box_bytes = plan.a_box_bytes, row_group = plan.row_group;
  const int i1 = plan.i1, out1 = plan.out1;     // output columns per tile
  TcGemmArgs g1;
  g1.C = h; g1.status = status; g1.ldc = c.d_ff;
  g1.tiles = mt == 2 ? tiles128 : tiles;          // always a list of 128-row tiles
  g1.n_tiles = mt == 2 ? n_tiles128 : n_tiles;
  g1.n_col_tiles = c.d_ff / out1;
  g1.k_blocks = c.d_model / kTcBK;
  g1.b_rows_per_phys = swiglu ? 2 * c.d_ff : c.d_ff;
  g1.b_rows_gate = swiglu ? c.d_ff : 0;
  g1.row_pair = nullptr; g1.gate = nullptr; g1.top_k = c.top_k;
  g1.row_group = row_group;
  g1.a_box_bytes = a_box_bytes;
  g1.early_b = 0;
  long long work = (long long)max_tiles * mt * g1.n_col_tiles;
  int grid = plan.grid;
  static const TcGemmKernel k1[2][3] = {
      {tc_gemm_kernel<256, kTcEpiReluBf16>, tc_gemm_kernel<128, kTcEpiReluBf16>, tc_gemm_kernel<64, kTcEpiReluBf16>},
      {tc_gemm_kernel<256, kTcEpiSwigluBf16>, tc_gemm_kernel<128, kTcEpiSwigluBf16>,
       tc_gemm_kernel<64, kTcEpiSwigluBf16>}};
  static const int smem1[3] = {TcSmem<256>::kBytes, TcSmem<128>::kBytes, TcSmem<64>::kBytes};
  if (s.only != 2) {
    if (launch_kernel(k1[swiglu ? 1 : 0][i1], dim3(grid), dim3(kTcThreads), smem1[i1], st, pdl, s.map_xp[ia], s.map_win[i1],
                      g1) != cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    ++*launches;
  }
  if (between) cudaEventRecord(between, st);
  if (s.only == 1) { *combined = scatter; return SWAPMOE_OK; }

  // ---- GEMM-2: y = h * W_out^T (or out = gate * y for top-1)
  const int i2 = mt == 2 ? 0 : tc_pick_bn(kBn2Options, 4, c.d_model, row_tiles_est, s.sm_count, a_box_bytes, 32);
  if (i2 < 0 || c.d_model % kBn2Options[i2]) return SWAPMOE_ERR_UNSUPPORTED;
  const int bn2 = kBn2Options[i2];
  TcGemmArgs g2;
  g2.C = scatter ? out : static_cast<void*>(y);
  g2.tiles = tiles; g2.n_tiles = n_tiles; g2.status = status; g2.ldc = c.d_model;
  g2.n_col_tiles = c.d_model / bn2;
  g2.k_blocks = c.d_ff / kTcBK;
  g2.b_rows_per_phys = c.d_model;
  g2.b_rows_gate = 0;
  g2.row_pair = row_pair; g2.gate = mgate; g2.top_k = c.top_k;
  g2.row_group = row_group;
  g2.a_box_bytes = a_box_bytes;
  g2.early_b = 1;
  work = (long long)max_tiles * g2.n_col_tiles;
  grid = work > s.sm_count ? s.sm_count : (int)work;
  const bool pdl2 = pdl && between == nullptr;
  static const TcGemmKernel k2[2][4] = {
      {tc_gemm_kernel<256, kTcEpiF32>, tc_gemm_kernel<128, kTcEpiF32>, tc_gemm_kernel<64, kTcEpiF32>,
       tc_gemm_kernel<32, kTcEpiF32>},
      {tc_gemm_kernel<256, kTcEpiScatterBf16>, tc_gemm_kernel<128, kTcEpiScatterBf16>,
       tc_gemm_kernel<64, kTcEpiScatterBf16>, tc_gemm_kernel<32, kTcEpiScatterBf16>}};
  static const int smem2[4] = {TcSmem<256>::kBytes, TcSmem<128>::kBytes, TcSmem<64>::kBytes, TcSmem<32>::kBytes};
  cudaError_t e;
  if (mt == 2) {
    const TcGemmKernel k = scatter ? tc_gemm_kernel<256, kTcEpiScatterBf16, 2> : tc_gemm_kernel<256, kTcEpiF32, 2>;
    e = launch_kernel(k, dim3(grid), dim3(kTcThreads), TcSmem<256, 2>::kBytes, st, pdl2, s.map_h[0], s.map_wout[0], g2);
  } else {
    e = launch_kernel(k2[scatter ? 1 : 0][i2], dim3(grid), dim3(kTcThreads), smem2[i2], st, pdl2, s.map_h[ia],
                      s.map_wout[i2], g2);
  }
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  ++*launches;
  *combined = scatter;
  return SWAPMOE_OK;
}

}  // namespace swapmoe
