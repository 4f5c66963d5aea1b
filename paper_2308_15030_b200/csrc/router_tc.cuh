// Router product on the tensor cores with the whole gate fused into its epilogue
// (SwapMoE Section 2: G(x); Fig. 4: Masked Gating; Eq. 1: importance terms).
//
// One CTA = tok (32, 64 or 128) tokens.  logits[tok, E] = x_tile * Wr^T is accumulated in TMEM
// by tcgen05.mma (bf16 -> fp32, M = 128: rows beyond tok are stale shared memory whose
// accumulator lanes are never read) from TMA-staged tiles; while the tiles stream through
// shared memory four warps accumulate ||x||^2 of their rows.  The logits then go TMEM ->
// shared memory and the gate runs with 256 / tok threads per token: half of them for the
// off-the-shelf gate, half for the masked gate (Fig. 4), each scanning its share of the
// experts; per-token candidates are merged in expert order so ties keep the lowest index.
// Small token tiles keep many SMs busy on small batches.  The last CTA to finish runs the
// slot scan.
#pragma once
#include "gemm_tc.cuh"
#include "permute.cuh"
#include "router_gate.cuh"
#include "gate_epilogue.cuh"

namespace swapmoe {

constexpr int kRtTok = 128;      // tokens per CTA
constexpr int kRtThreads = 256;

constexpr int kRtSmemBudget = 190 * 1024;

inline int router_tc_epad(int E) { return (E + 15) / 16 * 16; }
// tokens per CTA: every CTA re-reads the whole router matrix, so tiles shrink only for small
// batches (measured on B200: 32 and 64 tie at T = 2048, 64 beats 128 at T = 8192 by 5 us once
// the slot scan of the last CTA is cheap; 128-token tiles keep the grid within one wave beyond)
inline int router_tc_tok(int T) { return T <= 1024 ? 32 : (T <= 8192 ? 64 : 128); }
// A stage holds tok token rows and Epad router rows of one 64-column k-block.  (The MMA always
// reads 128 token rows: those beyond tok fall into neighbouring stage memory and only feed
// accumulator lanes that nobody reads.)
inline int router_tc_stage_bytes(int E, int tok) { return tok * kTcBK * 2 + router_tc_epad(E) * kTcBK * 2; }
constexpr int kRtMaxStages = 16;
inline int router_tc_stages(int E, int tok) {
  int s = (kRtSmemBudget - kRtTok * kTcBK * 2) / router_tc_stage_bytes(E, tok);
  return s > kRtMaxStages ? kRtMaxStages : s;
}
inline size_t router_tc_smem_bytes(int E, int tok) {
  // + one full 128-row tile of slack behind the stages for the MMA's over-read, and room for the
  // logits tile [tok][E+1] that later reuses the stage memory
  size_t stages = (size_t)router_tc_stages(E, tok) * router_tc_stage_bytes(E, tok) + kRtTok * kTcBK * 2;
  const size_t logit_tile = (size_t)tok * (E + 1) * 4;
  if (stages < logit_tile) stages = logit_tile;
  return stages + 2048 + 1024 + 8 * (2 * kRtMaxStages + 8) + 16 + gate_smem_bytes();
}

__global__ void __launch_bounds__(kRtThreads, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 const RouterArgs a, int32_t* status, int n_stages, int tok) {
  if ((int)blockIdx.x >= a.scan.n_cta) {
    // ---------------------------------------------------- weight-prefetch blocks
    pdl_wait();
    pdl_trigger();
    constexpr long long kChunk = 16384;
    const long long n_pf = (long long)(gridDim.x - a.scan.n_cta) * kRtThreads;
    const long long me = (long long)(blockIdx.x - a.scan.n_cta) * kRtThreads + threadIdx.x;
#pragma unroll 1
    for (int m = 0; m < 2; ++m) {
      const long long per_slot = a.pf_slot_bytes[m] / kChunk;
      const long long n_chunks = a.pf_total_bytes[m] / kChunk;
      for (long long c = me; c < n_chunks; c += n_pf) {
        const long long s = c / per_slot, o = c - s * per_slot;
        const char* src = a.pf_base[m] + (long long)a.pf_phys[s] * a.pf_slot_bytes[m] + o * kChunk;
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"((unsigned)kChunk) : "memory");
      }
    }
    return;
  }
  const int E = a.E;
  const int Epad = (E + 15) / 16 * 16;
  const int a_bytes = tok * kTcBK * 2, b_bytes = Epad * kTcBK * 2;   // token box, router box
  const int a_box_bytes = a_bytes;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  // layout: router tiles of all stages, then token tiles of all stages, then 16 KB of slack that
  // the 128-row MMA read of the last token tile may run into
  unsigned char* sB = smem;
  unsigned char* sA = smem + n_stages * b_bytes;
  float* slog = reinterpret_cast<float*>(smem);           // [tok][E+1], reuses the stage buffers
  const int stage_area = max(n_stages * (a_bytes + b_bytes) + kRtTok * kTcBK * 2, tok * (E + 1) * 4);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ((stage_area + 1023) & ~1023));
  uint64_t* full = bars;                  // [16]
  uint64_t* empty = bars + kRtMaxStages;  // [16]
  uint64_t* acc_full = bars + 2 * kRtMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kRtMaxStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const GateSmem g = gate_smem_carve(bars + 2 * kRtMaxStages + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * tok;
  const int k_blocks = a.d / kTcBK;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < Epad) tmem_cols <<= 1;

  if (tid == 0) {
    SWAPMOE_STAMP(0, 0);
    for (int s = 0; s < n_stages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 5); }
    ptx::mbar_init(acc_full, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmX);
    ptx::prefetch_tmap(&tmW);
  }
  if (warp == 2) {
    ptx::tmem_alloc(tmem_slot, tmem_cols);
    ptx::tmem_relinquish();
  }
  // The router matrix is a constant of the layer (no kernel writes it): the thread that initialised the barriers
  // requests its boxes for the first stages before the dependent-launch wait, and the token boxes right after it,
  // before the tables are staged.
  const int pre = k_blocks < n_stages ? k_blocks : n_stages;
  if (tid == 0) {
    for (int kb = 0; kb < pre; ++kb) {
      ptx::mbar_expect_tx(&full[kb], (uint32_t)(a_box_bytes + b_bytes));
      ptx::tma_load_2d(sB + kb * b_bytes, &tmW, &full[kb], kb * kTcBK, 0);
    }
    // ... and asks for its token boxes to be brought towards L2: a prefetch only moves DRAM contents into L2, where
    // later writes land too, so it cannot make the loads behind the wait see stale rows, and the first access to a
    // buffer is the slow one (2.9 us against 1.8 us for a box from DRAM)
    for (int kb = 0; kb < k_blocks; ++kb)
      asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(&tmX), "r"(kb * kTcBK), "r"(tok0)
                   : "memory");
  }
  pdl_wait();      // everything above touched only shared memory, TMEM, kernel parameters and the router matrix
  pdl_trigger();
  if (tid == 0) {
    SWAPMOE_STAMP(0, 1);
    for (int kb = 0; kb < pre; ++kb) ptx::tma_load_2d(sA + kb * a_bytes, &tmX, &full[kb], kb * kTcBK, tok0);
  }
  gate_load_tables(a, g);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // the first `pre` stages were requested above; the ring continues behind them
      int stage = pre == n_stages ? 0 : pre; uint32_t phase = pre == n_stages ? 1u : 0u;
      for (int kb = pre; kb < k_blocks; ++kb) {
        if (!bounded_wait(&empty[stage], phase ^ 1u, abort_flag, status, 11)) break;
        ptx::mbar_expect_tx(&full[stage], (uint32_t)(a_box_bytes + b_bytes));
        ptx::tma_load_2d(sA + stage * a_bytes, &tmX, &full[stage], kb * kTcBK, tok0);
        ptx::tma_load_2d(sB + stage * b_bytes, &tmW, &full[stage], kb * kTcBK, 0);
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
      }
      if (*abort_flag) {
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16(kRtTok, Epad);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int kb = 0; kb < k_blocks; ++kb) {
        ok = bounded_wait(&full[stage], phase, abort_flag, status, 12);
        if (!ok) break;
        ptx::tc_fence_after();
        if (kb == 0) SWAPMOE_STAMP(0, 2);
        const uint64_t da = make_kmajor_sw128_desc(ptx::smem_u32(sA + stage * a_bytes));
        const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(sB + stage * b_bytes));
#pragma unroll
        for (int kk = 0; kk < kTcBK / kTcUmmaK; ++kk)
          ptx::umma_bf16(tmem_base, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc,
                         (kb > 0 || kk > 0) ? 1u : 0u);
        ptx::umma_commit(&empty[stage]);
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
      }
      if (ok) ptx::umma_commit(acc_full);
      SWAPMOE_STAMP(0, 3);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------ ||x||^2 while the tiles stream through
    const int q = warp - 4, r = q * 32 + lane;
    const bool warp_has_rows = q * 32 < tok;       // whole warps beyond the token tile only keep the pipeline moving
    // eight independent partial sums: one accumulator would make the 64 FMAs of a k-block a dependent chain
    // (256 clocks), which bounded the whole main loop (0.55 us per k-block at d_model = 4096)
    float ss[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int stage = 0; uint32_t phase = 0;
    bool ok = true;
    for (int kb = 0; kb < k_blocks; ++kb) {
      ok = bounded_wait(&full[stage], phase, abort_flag, status, 13);
      if (!ok) break;
      if (warp_has_rows) {
        const uint4* row = reinterpret_cast<const uint4*>(sA + stage * a_bytes + r * 128);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          // the 16-byte chunks of a row may be visited in any order: rotate by the row
          // index so the threads of a quarter-warp hit different banks
          const uint4 u = row[(c + r) & 7];
          const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
            ss[2 * i] = fmaf(lo, lo, ss[2 * i]);
            ss[2 * i + 1] = fmaf(hi, hi, ss[2 * i + 1]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&empty[stage]);
      if (++stage == n_stages) { stage = 0; phase ^= 1u; }
    }
    if (warp_has_rows) g.snorm[r] = sqrtf(((ss[0] + ss[1]) + (ss[2] + ss[3])) + ((ss[4] + ss[5]) + (ss[6] + ss[7])));
    // ------------------------------------------------ logits: TMEM lane r -> shared-memory row r
    // (all MMAs have completed once acc_full fires, so the stage buffers are free to reuse)
    if (ok) ok = bounded_wait(acc_full, 0, abort_flag, status, 14);
    if (tid == 128) SWAPMOE_STAMP(0, 4);
    if (ok && warp_has_rows) {
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      float* srow = slog + (size_t)r * (E + 1);
      for (int c0 = 0; c0 < E; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld32(taddr + (uint32_t)c0, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c0 + i < E) srow[c0 + i] = __uint_as_float(v[i]);
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, tmem_cols);
  }
  if (tid == 0) SWAPMOE_STAMP(0, 5);
  const bool failed = *abort_flag != 0;
  // the stage memory is free again: the last CTA stages the scan inputs there
  gate_epilogue(a, g, slog, tok, tok0, failed, smem, stage_area);
}

}  // namespace swapmoe
