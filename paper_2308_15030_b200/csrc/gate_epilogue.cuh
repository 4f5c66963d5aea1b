// Gate of one token tile, shared by both router kernels (SwapMoE Section 2: G(x); Fig. 4:
// Masked Gating; Eq. 1: importance terms).  Input: the tile's logits in shared memory; output:
// both selections with their gate values, the slot of every pair, ||x||, and the CTA's partial
// sums for the slot scan.  256 threads; tok = 32, 64 or 128 tokens per CTA.
#pragma once
#include "common.cuh"
#include "permute.cuh"
#include "router_args.cuh"

namespace swapmoe {

constexpr int kGateTokMax = 128;   // largest token tile
constexpr int kGateThreads = 256;

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

// Shared-memory arrays of the gate, carved from one block by gate_smem_carve().
struct GateSmem {
  int* pe;             // [tok*k] unmasked expert per pair
  int* ps;             // [tok*k] slot per pair
  float* pt;           // [tok*k] Eq. (1) term per pair
  float* pm;           // [tok*k] Eq. (1) term under the masked routing
  float* snorm;        // [tok] ||x_t||
  int* s_e2s;          // [256] expert -> slot
  float* s_enorm;      // [256] ||E_e||
  uint32_t* s_mask;    // [2][8] valid / resident expert bits
  uint32_t* s_present; // [8] experts selected (unmasked) in this tile
  float* cand_v;       // [256 threads][kMaxTopK] per-thread top-k values
  int* cand_e;         //  ... and experts
  float* part_den;     // [256] partial softmax denominators
  float* s_m;          // [tok][2] row maximum per gate
};

__host__ __device__ constexpr size_t gate_smem_bytes() {
  return (size_t)4 * (4 * kGateTokMax * kMaxTopK + kGateTokMax + 2 * kMaxE + 24 +
                      2 * kGateThreads * kMaxTopK + kGateThreads + 2 * kGateTokMax);
}

__device__ __forceinline__ GateSmem gate_smem_carve(void* base) {
  GateSmem g;
  g.pe = static_cast<int*>(base);
  g.ps = g.pe + kGateTokMax * kMaxTopK;
  g.pt = reinterpret_cast<float*>(g.ps + kGateTokMax * kMaxTopK);
  g.pm = g.pt + kGateTokMax * kMaxTopK;
  g.snorm = g.pm + kGateTokMax * kMaxTopK;
  g.s_e2s = reinterpret_cast<int*>(g.snorm + kGateTokMax);
  g.s_enorm = reinterpret_cast<float*>(g.s_e2s + kMaxE);
  g.s_mask = reinterpret_cast<uint32_t*>(g.s_enorm + kMaxE);
  g.s_present = g.s_mask + 16;
  g.cand_v = reinterpret_cast<float*>(g.s_present + 8);
  g.cand_e = reinterpret_cast<int*>(g.cand_v + kGateThreads * kMaxTopK);
  g.part_den = reinterpret_cast<float*>(g.cand_e + kGateThreads * kMaxTopK);
  g.s_m = g.part_den + kGateThreads;
  return g;
}

// Copies the slot table and the expert norms into shared memory and builds the bit masks of
// valid and of resident experts.  All 256 threads; the caller synchronises afterwards.
__device__ __forceinline__ void gate_load_tables(const RouterArgs& a, const GateSmem& g) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // (a table entry outside [0, K) - possible only when the caller hands in its own table, as swapmoe_route_static
  // allows - counts as "not resident")
  for (int e = tid; e < kMaxE; e += kGateThreads) {
    const int sl = e < a.E ? a.e2s[e] : -1;
    g.s_e2s[e] = sl < a.K ? sl : -1;
    g.s_enorm[e] = e < a.E ? a.enorm[e] : 0.f;
  }
  // warp w builds word w of the valid-expert mask and of the resident-expert mask
  const int e = warp * 32 + lane;
  int sl = e < a.E ? a.e2s[e] : -1;
  if (sl >= a.K) sl = -1;
  const uint32_t wv = __ballot_sync(0xffffffffu, e < a.E), wr = __ballot_sync(0xffffffffu, sl >= 0);
  if (lane == 0) { g.s_mask[warp] = wv; g.s_mask[8 + warp] = wr; g.s_present[warp] = 0u; }
}

// The gate proper.  slog holds the tile's logits, row stride E + 1 floats (with at least 8
// floats readable behind the last row); g.snorm holds ||x_t|| of the tile's rows and
// gate_load_tables() has run, both made visible by a __syncthreads() in the caller.  When
// `failed` is set (the producer gave up on a bounded wait) zeros are written instead.
// scan_stage / scan_stage_bytes: shared memory that the last CTA may use to stage the scan
// inputs (may overlap slog).
//
// Thread t serves token t % tok.  Its group g = t / tok splits into the gate it evaluates
// (first half of the groups: off-the-shelf gate; second half: masked gate) and the share of
// the expert range it scans (whole 32-expert chunks, contiguous and ascending per share).
__device__ __forceinline__ void gate_epilogue(const RouterArgs& a, const GateSmem& g, const float* slog,
                                              int tok, int tok0, bool failed, void* scan_stage,
                                              int scan_stage_bytes) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int E = a.E, k = a.k;
  {
    // coalesced copy of the logits: a warp writes a token's row; four rows are in flight
    const int rows = min(tok, a.T - tok0);
    for (int t0 = warp * 4; t0 < rows; t0 += (kGateThreads / 32) * 4) {
      for (int e = lane; e < E; e += 32) {
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = slog[(size_t)min(t0 + q, tok - 1) * (E + 1) + e];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (t0 + q < rows) a.logits[(size_t)(tok0 + t0 + q) * E + e] = failed ? 0.f : v[q];
      }
    }
  }
  // tok is a power of two (32, 64, 128): shifts, not integer divisions, which cost dozens of
  // dependent instructions each in code that runs once
  const int tok_shift = 31 - __clz(tok);
  const int tl = tid & (tok - 1), grp = tid >> tok_shift;
  const int parts = (kGateThreads >> tok_shift) >> 1;       // threads per token and gate: 1, 2 or 4
  const bool masked = grp >= parts;
  const int part = masked ? grp - parts : grp;
  const int token = tok0 + tl;
  const float* row = slog + (size_t)tl * (E + 1);
  const uint32_t* allow = g.s_mask + (masked ? 8 : 0);
  const int n_chunks = (E + 31) >> 5, cpp = (n_chunks + parts - 1) >> (parts == 4 ? 2 : parts - 1);
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
    for (int j = 0; j < kMaxTopK; ++j) { g.cand_v[tid * kMaxTopK + j] = tk.v[j]; g.cand_e[tid * kMaxTopK + j] = tk.e[j]; }
  }
  __syncthreads();
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 6);
  // merge the shares of one (token, gate) in ascending expert order: a candidate only displaces
  // an entry it strictly beats, so equal logits keep the lowest expert index
  TopK fin;
  fin.init();
  if (part == 0) {
    for (int pp = 0; pp < parts; ++pp) {
      const int src = ((masked ? parts : 0) + pp) * tok + tl;
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j)
        if (j < k && g.cand_e[src * kMaxTopK + j] >= 0) fin.push(g.cand_v[src * kMaxTopK + j], g.cand_e[src * kMaxTopK + j], k);
    }
    g.s_m[tl * 2 + (masked ? 1 : 0)] = fin.v[0];
  }
  __syncthreads();
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 7);
  {
    const float m = g.s_m[tl * 2 + (masked ? 1 : 0)];
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
    g.part_den[tid] = den;
  }
  __syncthreads();
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 8);
  if (part == 0) {
    const float m = fin.v[0];
    float den = 0.f;
    if (a.renorm) {
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j)
        if (j < k) den += expf(fin.v[j] - m);
    } else {
      for (int pp = 0; pp < parts; ++pp) den += g.part_den[((masked ? parts : 0) + pp) * tok + tl];
    }
    const float xn = g.snorm[tl];
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) {
      if (j < k) {
        const int pl = tl * k + j;
        const size_t p = (size_t)token * k + j;
        const float gv = failed ? 0.f : expf(fin.v[j] - m) / den;
        const int e = fin.e[j];
        if (!masked) {
          if (token < a.T) {
            a.uidx[p] = e; a.ugate[p] = gv;
            g.pe[pl] = e; g.pt[pl] = xn * fabsf(gv) * g.s_enorm[e];   // one term of Eq. (1)
            atomicOr(&g.s_present[e >> 5], 1u << (e & 31));
          } else {
            g.pe[pl] = -1; g.pt[pl] = 0.f;
          }
        } else {
          if (token < a.T && e < 0) {
            // fewer resident experts than top_k (a caller-supplied table: the layer API rules it out): the pair
            // is routed nowhere instead of indexing the tables with -1
            a.midx[p] = -1; a.mgate[p] = 0.f; a.slot[p] = -1;
            g.ps[pl] = -1; g.pm[pl] = 0.f;
          } else if (token < a.T) {
            const int sl = g.s_e2s[e];
            a.midx[p] = e; a.mgate[p] = gv; a.slot[p] = sl;
            g.ps[pl] = sl; g.pm[pl] = xn * fabsf(gv) * g.s_enorm[e];
          } else {
            g.ps[pl] = -1; g.pm[pl] = 0.f;
          }
        }
      }
    }
    if (!masked && token < a.T) a.xnorm[token] = xn;
  }
  __syncthreads();
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 9);
  // Per-CTA partial sums with a fixed association (lane-strided partials, then the
  // shuffle tree), so the result does not depend on scheduling.  Only experts that some
  // token of this tile selected are visited; the others get an exact zero.
  const int npair = tok * k;
  for (int e = tid; e < E; e += kGateThreads) {
    a.cta_imp[(size_t)blockIdx.x * E + e] = 0.f;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + e] = 0.f;
  }
  for (int sl = tid; sl < a.K; sl += kGateThreads) a.cta_hist[(size_t)blockIdx.x * a.K + sl] = 0;
  __syncthreads();
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 10);
  for (int c = 0; c * 32 < E; ++c) {
    uint32_t present = g.s_present[c];
    for (int n = 0; present; ++n) {
      const int bit = __ffs(present) - 1;
      present &= present - 1;
      if ((n & 7) != warp) continue;                    // experts dealt round-robin to the warps
      const int e = c * 32 + bit;
      float sum = 0.f;
      int hits = 0;
      for (int p = lane; p < npair; p += 32) { sum += (g.pe[p] == e) ? g.pt[p] : 0.f; hits += (g.pe[p] == e); }
      sum = warp_sum(sum);
      hits = __reduce_add_sync(0xffffffffu, hits);
      if (lane == 0) {
        a.cta_imp[(size_t)blockIdx.x * E + e] = sum;
        if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + e] = (float)hits;
      }
    }
  }
  for (int sl = warp; sl < a.K; sl += kGateThreads / 32) {
    int c = 0;
    float m = 0.f;
    for (int p = lane; p < npair; p += 32) { c += (g.ps[p] == sl); m += (g.ps[p] == sl) ? g.pm[p] : 0.f; }
    c = __reduce_add_sync(0xffffffffu, c);
    m = warp_sum(m);
    if (lane == 0) {
      if (c) a.cta_hist[(size_t)blockIdx.x * a.K + sl] = c;
      if (a.cta_mimp) a.cta_mimp[(size_t)blockIdx.x * a.K + sl] = m;
    }
  }
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 11);
  finish_router_cta(a.scan, scan_stage, scan_stage_bytes);
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 12);
}

}  // namespace swapmoe
