// Router product, top-k gate, Masked Gating, slot remap and the per-token terms of
// the importance score (SwapMoE Section 2, Fig. 4, Eq. 1), CUDA-core version.
#pragma once
#include "common.cuh"
#include "permute.cuh"

namespace swapmoe {

struct RouterArgs {
  const void* x;            // [T, d] layer dtype
  const void* Wr;           // [E, d] layer dtype
  const float* ext_logits;  // [T, E] or nullptr
  const int32_t* e2s;       // [E] expert -> slot, -1 = not resident
  const float* enorm;       // [E]
  float* logits;            // [T, E]
  int32_t* uidx;            // [T, k]
  float* ugate;             // [T, k]
  int32_t* midx;            // [T, k]
  float* mgate;             // [T, k]
  int32_t* slot;            // [T, k]
  float* xnorm;             // [T]
  int32_t* cta_hist;        // [n_cta, K]
  float* cta_imp;           // [n_cta, E]
  float* cta_cnt;           // [n_cta, E] or nullptr
  float* cta_mimp;          // [n_cta, K] or nullptr
  int32_t T, d, E, k, K, renorm;
  ScanArgs scan;            // work of the last CTA to finish
  // Weight prefetch (tensor-core router only): blocks beyond the token tiles pull the resident
  // experts' matrices into L2 while the router runs, when HBM is otherwise idle.
  const char* pf_base[2];       // arena_in, arena_out
  long long pf_slot_bytes[2];   // bytes of one arena entry
  long long pf_total_bytes[2];  // bytes to prefetch, counted over logical slots 0..K-1 in order
  const int32_t* pf_phys;       // [K] arena entry of each logical slot
};

constexpr int kRouterDK = 32;  // contraction chunk staged in shared memory

// Selects the k largest of a token's logits that pass `allow_mask`, ties to the
// lowest expert index, and their gate values.  v[i] is the logit of expert
// lane + 32*i; allow_mask bit i says whether that expert may be chosen.
// Every lane returns the same sel_e / sel_g.
__device__ __forceinline__ void warp_topk_gate(const float (&v)[8], uint32_t allow_mask, int E, int k,
                                               int renorm, int lane, int (&sel_e)[kMaxTopK],
                                               float (&sel_g)[kMaxTopK]) {
  float sel_v[kMaxTopK];
  uint32_t avail = allow_mask;
  for (int j = 0; j < k; ++j) {
    float bv = -INFINITY;
    int be = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if ((avail >> i) & 1u) {
        if (be == 0x7fffffff || v[i] > bv) { bv = v[i]; be = lane + 32 * i; }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oe = __shfl_xor_sync(0xffffffffu, be, o);
      const bool take = (oe != 0x7fffffff) && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
      if (take) { bv = ov; be = oe; }
    }
    sel_e[j] = be;
    sel_v[j] = bv;
    if ((be & 31) == lane) avail &= ~(1u << (be >> 5));
  }
  const float m = sel_v[0];
  float den = 0.f;
  if (renorm) {
    for (int j = 0; j < k; ++j) den += expf(sel_v[j] - m);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if ((allow_mask >> i) & 1u) den += expf(v[i] - m);
    den = warp_sum(den);
  }
  for (int j = 0; j < k; ++j) sel_g[j] = expf(sel_v[j] - m) / den;
}

// Gate of one token, executed by a whole warp: v[i] = logit of expert lane + 32 i.
// Emits the unmasked and masked selections, the slot and the token's term of Eq. (1);
// tl is the token's index inside the CTA (pair arrays pe/ps/pt live in shared memory).
__device__ __forceinline__ void gate_token(const RouterArgs& a, const float (&v)[8], uint32_t valid_mask,
                                           uint32_t res_mask, int lane, int tok, int tl, float xn,
                                           int* pe, int* ps, float* pt, float* pm) {
  int ue[kMaxTopK], me[kMaxTopK];
  float ug[kMaxTopK], mg[kMaxTopK];
  warp_topk_gate(v, valid_mask, a.E, a.k, a.renorm, lane, ue, ug);   // off-the-shelf gate
  warp_topk_gate(v, res_mask, a.E, a.k, a.renorm, lane, me, mg);     // Masked Gating
  if (lane == 0) {
    for (int j = 0; j < a.k; ++j) {
      const int pl = tl * a.k + j;
      if (tok < a.T) {
        const int s = a.e2s[me[j]];
        const size_t p = (size_t)tok * a.k + j;
        a.uidx[p] = ue[j]; a.ugate[p] = ug[j];
        a.midx[p] = me[j]; a.mgate[p] = mg[j];
        a.slot[p] = s;
        pe[pl] = ue[j]; ps[pl] = s;
        pt[pl] = xn * fabsf(ug[j]) * a.enorm[ue[j]];   // one term of Eq. (1)
        pm[pl] = xn * fabsf(mg[j]) * a.enorm[me[j]];   // the same term under the masked routing
      } else {
        pe[pl] = -1; ps[pl] = -1; pt[pl] = 0.f; pm[pl] = 0.f;
      }
    }
    if (tok < a.T) a.xnorm[tok] = xn;
  }
}

// One CTA = kTokTile tokens; warp w owns tokens 4w..4w+3; lane l owns experts l+32i.
template <typename T>
__global__ void __launch_bounds__(256) router_gate_kernel(const RouterArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* xs = reinterpret_cast<float*>(smem_raw);              // [kTokTile][DK+1]
  float* ws = xs + kTokTile * (kRouterDK + 1);                 // [E][DK+1]
  int* pe = reinterpret_cast<int*>(ws + a.E * (kRouterDK + 1)); // [kTokTile*k] unmasked expert
  int* ps = pe + kTokTile * kMaxTopK;                           // [kTokTile*k] slot
  float* pt = reinterpret_cast<float*>(ps + kTokTile * kMaxTopK);  // importance term
  float* pm = pt + kTokTile * kMaxTopK;                            // importance term, masked routing

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tok0 = blockIdx.x * kTokTile;
  const T* x = static_cast<const T*>(a.x);
  const T* Wr = static_cast<const T*>(a.Wr);
  const int EI = (a.E + 31) >> 5;
  const bool have_ext = a.ext_logits != nullptr;

  float acc[4][8];
#pragma unroll
  for (int t = 0; t < 4; ++t)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[t][i] = 0.f;
  float sumsq = 0.f;
  pdl_wait();
  pdl_trigger();

  const int lrow = tid >> 3;         // token row this thread stages (0..31); == warp*4 + lane/8
  const int lcol = (tid & 7) * 4;    // 4 consecutive contraction indices
  const int ltok = tok0 + lrow;

  for (int c0 = 0; c0 < a.d; c0 += kRouterDK) {
    float xv[4] = {0.f, 0.f, 0.f, 0.f};
    if (ltok < a.T) load4(x + (size_t)ltok * a.d + c0 + lcol, xv);
    sumsq += xv[0] * xv[0] + xv[1] * xv[1] + xv[2] * xv[2] + xv[3] * xv[3];
    if (!have_ext) {
      __syncthreads();
#pragma unroll
      for (int q = 0; q < 4; ++q) xs[lrow * (kRouterDK + 1) + lcol + q] = xv[q];
      for (int v = tid; v < a.E * (kRouterDK / 4); v += 256) {
        const int e = v >> 3, c4 = (v & 7) * 4;
        float wv[4];
        load4(Wr + (size_t)e * a.d + c0 + c4, wv);
#pragma unroll
        for (int q = 0; q < 4; ++q) ws[e * (kRouterDK + 1) + c4 + q] = wv[q];
      }
      __syncthreads();
#pragma unroll 8
      for (int kk = 0; kk < kRouterDK; ++kk) {
        float xr[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) xr[t] = xs[(warp * 4 + t) * (kRouterDK + 1) + kk];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (i < EI) {
            const int e = lane + 32 * i;
            const float wv = (e < a.E) ? ws[e * (kRouterDK + 1) + kk] : 0.f;
#pragma unroll
            for (int t = 0; t < 4; ++t) acc[t][i] = fmaf(xr[t], wv, acc[t][i]);
          }
        }
      }
    }
  }
  // ||x||^2 of the 4 rows this warp staged: 8 consecutive lanes hold one row's partial sums.
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 1);
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 2);
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 4);

  uint32_t valid_mask = 0, res_mask = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int e = lane + 32 * i;
    if (e < a.E) {
      valid_mask |= 1u << i;
      if (a.e2s[e] >= 0) res_mask |= 1u << i;
    }
  }

#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int tl = warp * 4 + t;
    const int tok = tok0 + tl;
    const float xn = sqrtf(__shfl_sync(0xffffffffu, sumsq, t * 8));
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int e = lane + 32 * i;
      float lv = acc[t][i];
      if (have_ext && tok < a.T && e < a.E) lv = a.ext_logits[(size_t)tok * a.E + e];
      v[i] = lv;
      if (tok < a.T && e < a.E) a.logits[(size_t)tok * a.E + e] = lv;
    }
    gate_token(a, v, valid_mask, res_mask, lane, tok, tl, xn, pe, ps, pt, pm);
  }
  __syncthreads();
  // Per-CTA partial sums in a fixed order, so the result does not depend on scheduling.
  const int npair = kTokTile * a.k;
  for (int e = tid; e < a.E; e += 256) {
    float s = 0.f;
    int n = 0;
    for (int p = 0; p < npair; ++p) { s += (pe[p] == e) ? pt[p] : 0.f; n += (pe[p] == e); }
    a.cta_imp[(size_t)blockIdx.x * a.E + e] = s;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * a.E + e] = (float)n;
  }
  for (int s = tid; s < a.K; s += 256) {
    int c = 0;
    float m = 0.f;
    for (int p = 0; p < npair; ++p) { c += (ps[p] == s); m += (ps[p] == s) ? pm[p] : 0.f; }
    a.cta_hist[(size_t)blockIdx.x * a.K + s] = c;
    if (a.cta_mimp) a.cta_mimp[(size_t)blockIdx.x * a.K + s] = m;
  }
  finish_router_cta(a.scan);
}

inline size_t router_smem_bytes(int E) {
  return sizeof(float) * (kTokTile * (kRouterDK + 1) + (size_t)E * (kRouterDK + 1)) +
         (sizeof(int) * 2 + sizeof(float) * 2) * kTokTile * kMaxTopK;
}

}  // namespace swapmoe
