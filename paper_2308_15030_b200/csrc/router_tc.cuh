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

namespace swapmoe {

constexpr int kRtTok = 128;      // tokens per CTA
constexpr int kRtThreads = 256;

// Running top-k list, descending by value; a candidate is inserted below every entry
// that is >= it, so equal values stay in arrival (= expert index) order.
struct TopK {
  float v[kMaxTopK];
  int e[kMaxTopK];
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) { v[j] = -INFINITY; e[j] = -1; }
  }
  __device__ __forceinline__ void push(float cv, int ce, int k) {
    bool shifting = false;
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) {
      if (j < k && (shifting || e[j] < 0 || cv > v[j])) {
        const float tv = v[j]; const int te = e[j];
        v[j] = cv; e[j] = ce;
        cv = tv; ce = te;
        shifting = true;
      }
    }
  }
};
constexpr int kRtSmemBudget = 190 * 1024;

inline int router_tc_epad(int E) { return (E + 15) / 16 * 16; }
// tokens per CTA: every CTA re-reads the whole router matrix, so tiles shrink only for small
// batches (measured on B200: 64 is best at T = 2048, 128 at T = 8192)
inline int router_tc_tok(int T) { return T <= 1024 ? 32 : (T <= 4096 ? 64 : 128); }
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
  return stages + 2048 +
         (sizeof(int) * 2 + sizeof(float)) * kRtTok * kMaxTopK + sizeof(float) * kRtTok +
         (sizeof(int) + sizeof(float)) * kMaxE + sizeof(uint32_t) * 24 + 1024 + 8 * (2 * kRtMaxStages + 8) +
         (sizeof(float) + sizeof(int)) * kRtTok * 2 * 4 * kMaxTopK / 4 + sizeof(float) * kRtThreads + 1024 +
         sizeof(float) * kRtTok * kMaxTopK;
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
  const int E = a.E, k = a.k;
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
  int* pe = reinterpret_cast<int*>(bars + 2 * kRtMaxStages + 8);   // [tok*k] unmasked expert per pair
  int* ps = pe + kRtTok * kMaxTopK;                       // [tok*k] slot per pair
  float* pt = reinterpret_cast<float*>(ps + kRtTok * kMaxTopK);
  float* snorm = pt + kRtTok * kMaxTopK;                  // [tok] ||x_t||
  int* s_e2s = reinterpret_cast<int*>(snorm + kRtTok);    // [256] expert -> slot
  float* s_enorm = reinterpret_cast<float*>(s_e2s + kMaxE);   // [256] ||E_e||
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_enorm + kMaxE);  // [2][8] valid / resident bits
  uint32_t* s_present = s_mask + 16;                       // [8] experts selected (unmasked) in this tile
  float* cand_v = reinterpret_cast<float*>(s_present + 8); // [256 threads][kMaxTopK] per-thread top-k values
  int* cand_e = reinterpret_cast<int*>(cand_v + kRtThreads * kMaxTopK);   // ... and experts
  float* part_den = reinterpret_cast<float*>(cand_e + kRtThreads * kMaxTopK);   // [256] partial denominators
  float* s_m = part_den + kRtThreads;                      // [tok][2] row maximum per gate
  float* pm = s_m + 2 * kRtTok;                            // [tok*k] Eq. (1) term under the masked routing

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * tok;
  const int k_blocks = a.d / kTcBK;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < Epad) tmem_cols <<= 1;

  if (tid == 0) {
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
  pdl_wait();      // everything above touched only shared memory, TMEM and kernel parameters
  pdl_trigger();
  for (int e = tid; e < kMaxE; e += kRtThreads) {
    s_e2s[e] = e < E ? a.e2s[e] : -1;
    s_enorm[e] = e < E ? a.enorm[e] : 0.f;
  }
  {
    // warp w builds word w of the valid-expert mask and of the resident-expert mask
    const int e = warp * 32 + lane;
    const int sl = e < E ? a.e2s[e] : -1;
    const uint32_t wv = __ballot_sync(0xffffffffu, e < E), wr = __ballot_sync(0xffffffffu, sl >= 0);
    if (lane == 0) { s_mask[warp] = wv; s_mask[8 + warp] = wr; s_present[warp] = 0u; }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int kb = 0; kb < k_blocks; ++kb) {
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
    }
  } else if (warp >= 4) {
    // ------------------------------------------------ ||x||^2 while the tiles stream through
    const int q = warp - 4, r = q * 32 + lane;
    const bool warp_has_rows = q * 32 < tok;       // whole warps beyond the token tile only keep the pipeline moving
    float sumsq = 0.f;
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
            sumsq = fmaf(lo, lo, sumsq);
            sumsq = fmaf(hi, hi, sumsq);
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&empty[stage]);
      if (++stage == n_stages) { stage = 0; phase ^= 1u; }
    }
    if (warp_has_rows) snorm[r] = sqrtf(sumsq);
    // ------------------------------------------------ logits: TMEM lane r -> shared-memory row r
    // (all MMAs have completed once acc_full fires, so the stage buffers are free to reuse)
    if (ok) ok = bounded_wait(acc_full, 0, abort_flag, status, 14);
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
  const bool failed = *abort_flag != 0;
  {
    // coalesced copy of the logits: a warp writes a token's row; four rows are in flight
    const int rows = min(tok, a.T - tok0);
    for (int t0 = warp * 4; t0 < rows; t0 += (kRtThreads / 32) * 4) {
      for (int e = lane; e < E; e += 32) {
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = slog[(size_t)(t0 + q) * (E + 1) + e];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (t0 + q < rows) a.logits[(size_t)(tok0 + t0 + q) * E + e] = failed ? 0.f : v[q];
      }
    }
  }
  // ---------------------------------------------------- gate: 256 / tok threads per token
  // Thread t serves token t % tok.  Its group g = t / tok splits into the gate it evaluates
  // (first half of the groups: off-the-shelf gate; second half: masked gate) and the share of
  // the expert range it scans (whole 32-expert chunks, contiguous and ascending per share).
  const int tl = tid % tok, grp = tid / tok;
  const int parts = (kRtThreads / tok) >> 1;                // threads per token and gate: 1, 2 or 4
  const bool masked = grp >= parts;
  const int part = masked ? grp - parts : grp;
  const int token = tok0 + tl;
  const float* row = slog + (size_t)tl * (E + 1);
  const uint32_t* allow = s_mask + (masked ? 8 : 0);
  const int n_chunks = (E + 31) >> 5, cpp = (n_chunks + parts - 1) / parts;
  const int e_lo = min(E, part * cpp * 32), e_hi = min(E, (part + 1) * cpp * 32);
  {
    // The loops below run once per CTA, so they are kept rolled (short bodies that stay in the
    // instruction cache) rather than unrolled over the whole expert range.
    TopK tk;
    tk.init();
    if (k == 1) {
      float best = -INFINITY;
      int bi = -1;
#pragma unroll 4
      for (int e = e_lo; e < e_hi; ++e) {
        const float l = row[e];
        const bool take = ((allow[e >> 5] >> (e & 31)) & 1u) && (bi < 0 || l > best);
        best = take ? l : best;
        bi = take ? e : bi;
      }
      tk.v[0] = best;
      tk.e[0] = bi;
    } else {
      float thr = -INFINITY;
      int filled = 0;
#pragma unroll 1
      for (int e = e_lo; e < e_hi; ++e) {
        const float l = row[e];
        if (((allow[e >> 5] >> (e & 31)) & 1u) && (filled < k || l > thr)) {
          tk.push(l, e, k);
          ++filled;
          thr = (k == 2) ? tk.v[1] : (k == 3) ? tk.v[2] : tk.v[3];
        }
      }
    }
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) { cand_v[tid * kMaxTopK + j] = tk.v[j]; cand_e[tid * kMaxTopK + j] = tk.e[j]; }
  }
  __syncthreads();
  // merge the shares of one (token, gate) in ascending expert order: a candidate only displaces
  // an entry it strictly beats, so equal logits keep the lowest expert index
  TopK fin;
  fin.init();
  if (part == 0) {
    for (int pp = 0; pp < parts; ++pp) {
      const int src = ((masked ? parts : 0) + pp) * tok + tl;
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j)
        if (j < k && cand_e[src * kMaxTopK + j] >= 0) fin.push(cand_v[src * kMaxTopK + j], cand_e[src * kMaxTopK + j], k);
    }
    s_m[tl * 2 + (masked ? 1 : 0)] = fin.v[0];
  }
  __syncthreads();
  {
    const float m = s_m[tl * 2 + (masked ? 1 : 0)];
    float den = 0.f;
    if (!a.renorm) {
      // eight interleaved partial sums: short dependency chains and a tree-shaped total
      float acc8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
      for (int e0 = e_lo; e0 < e_hi; e0 += 8) {
        const uint32_t w = allow[e0 >> 5] >> (e0 & 31);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float t = __expf(row[e0 + i] - m);
          acc8[i] += ((w >> i) & 1u) ? t : 0.f;
        }
      }
      den = ((acc8[0] + acc8[1]) + (acc8[2] + acc8[3])) + ((acc8[4] + acc8[5]) + (acc8[6] + acc8[7]));
    }
    part_den[tid] = den;
  }
  __syncthreads();
  if (part == 0) {
    const float m = fin.v[0];
    float den = 0.f;
    if (a.renorm) {
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j)
        if (j < k) den += expf(fin.v[j] - m);
    } else {
      for (int pp = 0; pp < parts; ++pp) den += part_den[((masked ? parts : 0) + pp) * tok + tl];
    }
    const float xn = snorm[tl];
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) {
      if (j < k) {
        const int pl = tl * k + j;
        const size_t p = (size_t)token * k + j;
        const float g = failed ? 0.f : expf(fin.v[j] - m) / den;
        const int e = fin.e[j];
        if (!masked) {
          if (token < a.T) {
            a.uidx[p] = e; a.ugate[p] = g;
            pe[pl] = e; pt[pl] = xn * fabsf(g) * s_enorm[e];   // one term of Eq. (1)
            atomicOr(&s_present[e >> 5], 1u << (e & 31));
          } else {
            pe[pl] = -1; pt[pl] = 0.f;
          }
        } else {
          if (token < a.T) {
            const int sl = s_e2s[e];
            a.midx[p] = e; a.mgate[p] = g; a.slot[p] = sl;
            ps[pl] = sl; pm[pl] = xn * fabsf(g) * s_enorm[e];
          } else {
            ps[pl] = -1; pm[pl] = 0.f;
          }
        }
      }
    }
    if (!masked && token < a.T) a.xnorm[token] = xn;
  }
  __syncthreads();
  // Per-CTA partial sums with a fixed association (lane-strided partials, then the
  // shuffle tree), so the result does not depend on scheduling.  Only experts that some
  // token of this tile selected are visited; the others get an exact zero.
  const int npair = tok * k;
  for (int e = tid; e < E; e += kRtThreads) {
    a.cta_imp[(size_t)blockIdx.x * E + e] = 0.f;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + e] = 0.f;
  }
  for (int sl = tid; sl < a.K; sl += kRtThreads) a.cta_hist[(size_t)blockIdx.x * a.K + sl] = 0;
  __syncthreads();
  for (int c = 0; c * 32 < E; ++c) {
    uint32_t present = s_present[c];
    for (int n = 0; present; ++n) {
      const int bit = __ffs(present) - 1;
      present &= present - 1;
      if ((n & 7) != warp) continue;                    // experts dealt round-robin to the warps
      const int e = c * 32 + bit;
      float sum = 0.f;
      int hits = 0;
      for (int p = lane; p < npair; p += 32) { sum += (pe[p] == e) ? pt[p] : 0.f; hits += (pe[p] == e); }
      sum = warp_sum(sum);
      hits = __reduce_add_sync(0xffffffffu, hits);
      if (lane == 0) {
        a.cta_imp[(size_t)blockIdx.x * E + e] = sum;
        if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + e] = (float)hits;
      }
    }
  }
  for (int sl = warp; sl < a.K; sl += kRtThreads / 32) {
    int c = 0;
    float m = 0.f;
    for (int p = lane; p < npair; p += 32) { c += (ps[p] == sl); m += (ps[p] == sl) ? pm[p] : 0.f; }
    c = __reduce_add_sync(0xffffffffu, c);
    m = warp_sum(m);
    if (lane == 0) {
      if (c) a.cta_hist[(size_t)blockIdx.x * a.K + sl] = c;
      if (a.cta_mimp) a.cta_mimp[(size_t)blockIdx.x * a.K + sl] = m;
    }
  }
  finish_router_cta(a.scan, smem, stage_area);      // the stage memory is free again: stage the scan inputs there
}

}  // namespace swapmoe
