// Router, both gates and the per-CTA partial sums for small batches (bf16, up to 64 tokens),
// SwapMoE Section 2 (G(x)), Fig. 4 (Masked Gating), Eq. 1 (importance terms).
//
// The tcgen05 router spends 20 us of fixed cost (TMEM hand-offs, a gate written for 32-128 token
// tiles) on a handful of tokens.  Here a CTA takes EIGHT tokens and routes them the way the
// one-launch decode kernel does: the router matrix arrives in two TMA wave buffers (requested
// before the wait on the predecessor), the product is warp-level mma with the eight tokens as the
// eight mma columns and the contraction split over 16 warps, and a warp computes a token's gate.
// The outputs, the per-CTA partial sums and the last CTA's slot scan are those of the other
// routers, so the permutation and the grouped GEMMs that follow are unchanged.
#pragma once
#include "common.cuh"
#include "decode_fused.cuh"
#include "permute.cuh"
#include "router_args.cuh"

namespace swapmoe {

constexpr int kRsTok = kDecMaxTokens;     // tokens per CTA
constexpr int kRsMaxTokens = 64;          // batches up to this size take this router

struct RsSmem {
  int xs, slog, red, route, bars, pairs, total;
};
__host__ __device__ inline RsSmem router_small_layout(int d) {
  RsSmem m;
  int o = 2 * kDecHalfBytes;
  m.xs = o;    o += kRsTok * (d * 2 + kDecRowPad);
  m.slog = o;  o += kRsTok * (kMaxE + 1) * 4;
  o = (o + 15) & ~15;
  m.red = o;   o += kDecWarps * 32 * 8 * 4;
  m.route = o; o += (int)sizeof(DecRoute);
  o = (o + 15) & ~15;
  m.bars = o;  o += 16;
  m.pairs = o; o += kDecMaxPairs * 2 * 4;   // Eq. (1) terms per pair: unmasked, masked
  m.total = o;
  return m;
}
inline size_t router_small_smem_bytes(int d) { return (size_t)router_small_layout(d).total + 1024; }

__global__ void __launch_bounds__(kDecThreads, 1) router_small_kernel(const RouterArgs a, int32_t* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int d = a.d, E = a.E, k = a.k, K = a.K;
  const int chunks = d / 8, pitch = d * 2 + kDecRowPad;
  const RsSmem lay = router_small_layout(d);
  unsigned char* ring = smem;
  unsigned char* xs = smem + lay.xs;
  float* slog = reinterpret_cast<float*>(smem + lay.slog);
  float* red = reinterpret_cast<float*>(smem + lay.red);
  DecRoute* R = reinterpret_cast<DecRoute*>(smem + lay.route);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + lay.bars);
  float* pt = reinterpret_cast<float*>(smem + lay.pairs);   // [pairs] Eq. (1) term, off-the-shelf routing
  float* pm = pt + kDecMaxPairs;                            // [pairs] ... masked routing
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * kRsTok;
  const int T = min(kRsTok, a.T - tok0);                    // tokens of this CTA
  const int P = T * k;
  const bf16* x = static_cast<const bf16*>(a.x) + (size_t)tok0 * d;
  const bf16* Wr = static_cast<const bf16*>(a.Wr);

  const int RW = decode_rows_per_wave(d);
  const int n_rw = (E + RW - 1) / RW;
  auto issue_router_wave = [&](int w) {                     // all of warp 0
    const int rows = min(RW, E - w * RW);
    uint64_t* bar = &bars[w & 1];
    if (lane == 0) ptx::mbar_expect_tx(bar, (uint32_t)(rows * d * 2));
    __syncwarp();
    if (lane < rows)
      ptx::bulk_load_1d(ring + (w & 1) * kDecHalfBytes + lane * pitch, Wr + ((size_t)w * RW + lane) * d, (uint32_t)(d * 2), bar);
  };
  if (tid == 0) {
    ptx::mbar_init(&bars[0], 1);
    ptx::mbar_init(&bars[1], 1);
    R->abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (warp == 0) {                                          // the router matrix is a constant of the layer
    issue_router_wave(0);
    if (n_rw > 1) issue_router_wave(1);
  }
  pdl_wait();
  pdl_trigger();
  {
    const int t = warp & (kRsTok - 1);                      // token t is copied by warps t and t + 8
    if (t < T) {
#pragma unroll 1
      for (int c0 = (warp >> 3) * 32 + lane; c0 < chunks; c0 += 256) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 64 * u < chunks) v[u] = reinterpret_cast<const uint4*>(x)[t * chunks + c0 + 64 * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 64 * u < chunks) *reinterpret_cast<uint4*>(xs + t * pitch + (c0 + 64 * u) * 16) = v[u];
      }
    }
  }
  if (tid < kMaxE) R->e2s[tid] = tid < E ? a.e2s[tid] : -1;
  if (tid < kRsTok) R->tok[tid] = min(tid, T - 1);
  __syncthreads();
  if (warp < T) {
    float ss = 0.f;
#pragma unroll 1
    for (int c = lane; c < chunks; c += 32) {
      const uint4 u = *reinterpret_cast<const uint4*>(xs + warp * pitch + c * 16);
      const uint32_t w4[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w4[i] << 16), hi = __uint_as_float(w4[i] & 0xFFFF0000u);
        ss = fmaf(lo, lo, ss);
        ss = fmaf(hi, hi, ss);
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) R->xn[warp] = sqrtf(ss);
  }
  bool alive = true;
#pragma unroll 1
  for (int w = 0; w < n_rw; ++w) {
    if (!dec_wait_wave(bars, w, R, status, 23)) { alive = false; break; }
    dec_wave_dots(ring + (w & 1) * kDecHalfBytes, min(RW, E - w * RW), d, xs, R, T, red, slog + w * RW, kMaxE + 1);
    if (warp == 0 && w + 2 < n_rw) {
      ptx::fence_proxy_async();
      issue_router_wave(w + 2);
    }
  }
  __syncthreads();
  if (warp < 2 * kRsTok && (warp & (kRsTok - 1)) < T) {
    // gate of token (warp & 7): warps 0-7 the off-the-shelf gate, 8-15 the masked one
    const int t = warp & (kRsTok - 1), pass = warp / kRsTok;
    float v[8];
    uint32_t allow = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int e = lane + 32 * i;
      v[i] = (e < E && alive) ? slog[t * (kMaxE + 1) + e] : (e < E ? 0.f : -INFINITY);
      if (e < E && (pass == 0 || R->e2s[e] >= 0)) allow |= 1u << i;
    }
    int se[kMaxTopK];
    float sg[kMaxTopK];
    dec_topk_gate(v, allow, k, a.renorm, lane, se, sg);
    if (lane == 0) {
      const float xn = R->xn[t];
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j) {
        if (j < k) {
          const int p = t * k + j;
          const size_t gp = (size_t)(tok0 + t) * k + j;
          const float gv = alive ? sg[j] : 0.f;
          if (pass == 0) {
            R->ue[p] = se[j];
            a.uidx[gp] = se[j]; a.ugate[gp] = gv;
            pt[p] = xn * fabsf(gv) * a.enorm[se[j]];
          } else {
            const int sl = R->e2s[se[j]];
            R->sl[p] = sl;
            a.midx[gp] = se[j]; a.mgate[gp] = gv; a.slot[gp] = sl;
            pm[p] = xn * fabsf(gv) * a.enorm[se[j]];
          }
        }
      }
      if (pass == 0) a.xnorm[tok0 + t] = xn;
    }
  }
#pragma unroll 1
  for (int i = tid; i < T * E; i += kDecThreads) {
    const int t = i / E, e = i - t * E;
    a.logits[(size_t)(tok0 + t) * E + e] = alive ? slog[t * (kMaxE + 1) + e] : 0.f;
  }
  __syncthreads();
  // per-CTA partial sums in pair order (at most 32 pairs): fixed order, run to run
  if (tid < E) {
    float s = 0.f;
    int n = 0;
#pragma unroll 1
    for (int p = 0; p < P; ++p)
      if (R->ue[p] == tid) { s += pt[p]; ++n; }
    a.cta_imp[(size_t)blockIdx.x * E + tid] = s;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + tid] = (float)n;
  }
  if (tid >= kDecThreads - K) {
    const int sl = kDecThreads - 1 - tid;                   // the last K threads: slot sums
    int c = 0;
    float m = 0.f;
#pragma unroll 1
    for (int p = 0; p < P; ++p)
      if (R->sl[p] == sl) { ++c; m += pm[p]; }
    a.cta_hist[(size_t)blockIdx.x * K + sl] = c;
    if (a.cta_mimp) a.cta_mimp[(size_t)blockIdx.x * K + sl] = m;
  }
  if (!alive && tid == 0) {
    // a wait gave up: let copies that may still be in flight land before the buffers are reused
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  finish_router_cta(a.scan, ring, 2 * kDecHalfBytes);       // the wave buffers are free: stage the scan inputs there
}

}  // namespace swapmoe
