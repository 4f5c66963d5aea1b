// Router, both gates and the per-CTA partial sums for small batches (bf16, up to 64 tokens),
// SwapMoE Section 2 (G(x)), Fig. 4 (Masked Gating), Eq. 1 (importance terms).
//
// The tcgen05 router spends 20 us of fixed cost (TMEM hand-offs, a gate written for 32-128 token
// tiles) on a handful of tokens.  Here a CTA takes eight or sixteen tokens and routes them the way the
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

constexpr int kRsTok = kDecMaxTokens;     // tokens per mma column tile
constexpr int kRsMaxNT = 2;               // column tiles (of eight tokens) per CTA: 1 or 2
constexpr int kRsMaxPairs = kRsTok * kRsMaxNT * kMaxTopK;
constexpr int kRsMaxTokens = 64;          // batches up to this size use eight-token CTAs

// Routing state of one CTA's tokens (shared memory).
struct RsRoute {
  int ue[kRsMaxPairs], sl[kRsMaxPairs];   // off-the-shelf expert and slot per pair p = t*k + j
  float pt[kRsMaxPairs], pm[kRsMaxPairs]; // Eq. (1) term per pair: off-the-shelf routing, masked routing
  float xn[kRsTok * kRsMaxNT];
  float enorm[kMaxE];                      // ||E_e|| of every expert (the gate tasks would otherwise wait for a global load each)
};

struct RsSmem {
  int xs, slog, red, route, bars, pairs, total;
};
__host__ __device__ inline RsSmem router_small_layout(int d, int nt) {
  RsSmem m;
  int o = 2 * kDecHalfBytes;
  m.xs = o;    o += kRsTok * nt * (d * 2 + kDecRowPad);
  m.slog = o;  o += kRsTok * nt * (kMaxE + 1) * 4;
  o = (o + 15) & ~15;
  m.red = o;   o += kDecWarps * 32 * 8 * 4 * nt;
  m.route = o; o += (int)sizeof(DecRoute);
  o = (o + 15) & ~15;
  m.bars = o;  o += 16;
  m.pairs = o; o += (int)sizeof(RsRoute);
  m.total = o;
  return m;
}
inline size_t router_small_smem_bytes(int d, int nt) { return (size_t)router_small_layout(d, nt).total + 1024; }

// dst[(8 j + n) * dst_stride + r] = <row r of the wave buffer, token 8 j + n> for r < rows <= 32, j < NT,
// 8 j + n < n_tok: dec_wave_dots for NT column tiles at once (the weight fragments are loaded once).
template <int NT>
__device__ __forceinline__ void rs_wave_dots(const unsigned char* st, int rows, int d, const unsigned char* xs,
                                             int n_tok, float* red, float* dst, int dst_stride) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int pitch = d * 2 + kDecRowPad;
  float acc[2][NT][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[i][j][q] = 0.f;
  // (row indices beyond what a wave buffer holds at this row length are clamped to its last row: their products
  // are dropped, and no read leaves the buffer)
  const int rmax = decode_rows_per_wave(d) - 1;
  const unsigned char* ar[2][2];               // rows 16 i + 8 h + g of the buffer
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h) ar[i][h] = st + min(16 * i + 8 * h + g, rmax) * pitch + t * 4;
#pragma unroll 2
  for (int ks = warp; ks < d / 16; ks += kDecWarps) {
    const int kb = ks * 32;
    uint32_t b0[NT], b1[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const unsigned char* xrow = xs + min(8 * j + g, n_tok - 1) * pitch + t * 4 + kb;
      b0[j] = lds32(xrow);
      b1[j] = lds32(xrow + 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint32_t a0 = lds32(ar[i][0] + kb), a1 = lds32(ar[i][1] + kb), a2 = lds32(ar[i][0] + kb + 16),
                     a3 = lds32(ar[i][1] + kb + 16);
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_bf16_16x8x16(acc[i][j], a0, a1, a2, a3, b0[j], b1[j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      float* rp = red + ((warp * NT + j) * 32 + i * 16 + g) * 8 + 2 * t;
      *reinterpret_cast<float2*>(rp) = make_float2(acc[i][j][0], acc[i][j][1]);
      *reinterpret_cast<float2*>(rp + 8 * 8) = make_float2(acc[i][j][2], acc[i][j][3]);
    }
  __syncthreads();
  if (tid < 32 * 8 * NT) {
    const int j = tid >> 8, r = (tid >> 3) & 31, n = tid & 7;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) s += red[((w * NT + j) * 32 + r) * 8 + n];
    if (r < rows && 8 * j + n < n_tok) dst[(8 * j + n) * dst_stride + r] = s;
  }
  __syncthreads();
}

// All logits of the CTA in ONE pass when the router matrix fits the two wave buffers (E <= 2 waves of rows):
// a warp owns a tile of 16 experts (all NT token tiles of it: the router-matrix fragments are read once and
// feed NT mma) and a contiguous share of the contraction; the 16 / tiles shares of a tile are added in order.
// Per CTA that is one pair of barriers and a 4-way sum for 64 experts x 16 tokens, where the wave-by-wave form
// (every wave's contraction split over all 16 warps) pays a 16-way sum and two barriers per wave.
// slog[token * (kMaxE + 1) + expert] receives the logits.
template <int NT>
__device__ __forceinline__ void rs_dots_resident(const unsigned char* ring, int E, int RW, int d, const unsigned char* xs,
                                                 int n_tok, float* red, float* slog) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int pitch = d * 2 + kDecRowPad;
  const int MT = (E + 15) >> 4;                 // 16-expert row tiles (<= 4)
  int tiles_p2 = 1;
  while (tiles_p2 < MT) tiles_p2 <<= 1;
  const int S = kDecWarps / tiles_p2;           // shares of the contraction per tile (>= 4)
  const int m = warp & (tiles_p2 - 1), part = warp / tiles_p2;
  if (m < MT) {
    const int row0 = m * 16;                    // first expert of the tile; wave row0 / RW, row row0 % RW inside it
    const unsigned char* ap0 = ring + (row0 / RW) * kDecHalfBytes + ((row0 % RW) + g) * pitch + t * 4;
    const unsigned char* xrow[NT];
#pragma unroll
    for (int j = 0; j < NT; ++j) xrow[j] = xs + min(8 * j + g, n_tok - 1) * pitch + t * 4;
    const int nks = d / 16, ks0 = part * nks / S, ks1 = (part + 1) * nks / S;
    float acc[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[j][q] = 0.f;
#pragma unroll 4
    for (int ks = ks0; ks < ks1; ++ks) {
      const int kb = ks * 32;
      const uint32_t a0 = lds32(ap0 + kb), a1 = lds32(ap0 + 8 * pitch + kb), a2 = lds32(ap0 + kb + 16),
                     a3 = lds32(ap0 + 8 * pitch + kb + 16);
#pragma unroll
      for (int j = 0; j < NT; ++j) {            // NT independent accumulators: NT chains of dependent mma
        const uint32_t b0 = lds32(xrow[j] + kb), b1 = lds32(xrow[j] + kb + 16);
        mma_bf16_16x8x16(acc[j], a0, a1, a2, a3, b0, b1);
      }
    }
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      float* rp = red + (((part * MT + m) * NT + j) * 16 + g) * 8 + 2 * t;
      *reinterpret_cast<float2*>(rp) = make_float2(acc[j][0], acc[j][1]);
      *reinterpret_cast<float2*>(rp + 8 * 8) = make_float2(acc[j][2], acc[j][3]);
    }
  }
  if (tid == 0) SWAPMOE_STAMP(0, 12);
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 13);
  const int n_tiles = MT * NT;
  for (int o = tid; o < n_tiles * 128; o += kDecThreads) {
    const int tl = o >> 7, r = (o >> 3) & 15, c = o & 7;      // tl = m * NT + j
    float sum = 0.f;
    for (int p = 0; p < S; ++p) sum += red[((p * n_tiles + tl) * 16 + r) * 8 + c];
    const int mm = tl / NT, j = tl - mm * NT;
    const int e = mm * 16 + r, tok = 8 * j + c;
    if (e < E && tok < n_tok) slog[tok * (kMaxE + 1) + e] = sum;
  }
  __syncthreads();
}

template <int NT>
__global__ void __launch_bounds__(kDecThreads, 1) router_small_kernel(const RouterArgs a, int32_t* status) {
  constexpr int TOK = kRsTok * NT;                          // tokens per CTA
  if ((int)blockIdx.x >= a.scan.n_cta) {                    // blocks beyond the token tiles prefetch weights
    pdl_wait();
    pdl_trigger();
    router_prefetch_role(a, a.scan.n_cta);
    return;
  }
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 0);
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int d = a.d, E = a.E, k = a.k, K = a.K;
  const int chunks = d / 8, pitch = d * 2 + kDecRowPad;
  const RsSmem lay = router_small_layout(d, NT);
  unsigned char* ring = smem;
  unsigned char* xs = smem + lay.xs;
  float* slog = reinterpret_cast<float*>(smem + lay.slog);
  float* red = reinterpret_cast<float*>(smem + lay.red);
  DecRoute* R = reinterpret_cast<DecRoute*>(smem + lay.route);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + lay.bars);
  RsRoute* Q = reinterpret_cast<RsRoute*>(smem + lay.pairs);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tok0 = blockIdx.x * TOK;
  const int T = min(TOK, a.T - tok0);                       // tokens of this CTA
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
  if (warp == 1 && lane == 0) {
    // The CTA's token rows (one contiguous range) are pulled towards L2 while the kernel in front still runs.
    // A prefetch only moves what DRAM holds into L2, where any later write of the producer lands too, so it
    // cannot make the loads after the wait see stale data; it saves them the DRAM latency when x is cold.
    const uint32_t bytes = (uint32_t)(T * d * 2);
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(x), "r"(bytes) : "memory");
  }
  pdl_wait();
  pdl_trigger();
  if (tid == 0) SWAPMOE_STAMP(0, 1);
  {
    // token t is copied by the kDecWarps / TOK warps t, t + TOK, ...; four independent loads per lane and round
    constexpr int kWpt = kDecWarps / TOK;                   // warps per token: 2 or 1
    const int t = warp & (TOK - 1);
    if (t < T) {
#pragma unroll 1
      for (int c0 = (warp / TOK) * 32 + lane; c0 < chunks; c0 += 128 * kWpt) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 32 * kWpt * u < chunks) v[u] = reinterpret_cast<const uint4*>(x)[t * chunks + c0 + 32 * kWpt * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 32 * kWpt * u < chunks) *reinterpret_cast<uint4*>(xs + t * pitch + (c0 + 32 * kWpt * u) * 16) = v[u];
      }
    }
  }
  if (tid < kMaxE) {
    R->e2s[tid] = tid < E ? a.e2s[tid] : -1;
    Q->enorm[tid] = tid < E ? a.enorm[tid] : 0.f;
  }
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
    if (lane == 0) Q->xn[warp] = sqrtf(ss);
  }
  if (tid == 0) SWAPMOE_STAMP(0, 2);
  bool alive = true;
  if (n_rw <= 2 && RW % 16 == 0) {
    // the whole router matrix is resident in the two wave buffers: one pass over all experts
    for (int w = 0; w < n_rw && alive; ++w) alive = dec_wait_wave(bars, w, R, status, 23);
    if (tid == 0) SWAPMOE_STAMP(0, 11);
    if (alive) rs_dots_resident<NT>(ring, E, RW, d, xs, T, red, slog);
  } else {
#pragma unroll 1
    for (int w = 0; w < n_rw; ++w) {
      if (!dec_wait_wave(bars, w, R, status, 23)) { alive = false; break; }
      rs_wave_dots<NT>(ring + (w & 1) * kDecHalfBytes, min(RW, E - w * RW), d, xs, T, red, slog + w * RW, kMaxE + 1);
      if (warp == 0 && w + 2 < n_rw) {
        ptx::fence_proxy_async();
        issue_router_wave(w + 2);
      }
    }
  }
  if (!alive)
    for (int i = tid; i < TOK * (kMaxE + 1); i += kDecThreads) slog[i] = 0.f;
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 3);
  if constexpr (NT == 2) {
    // sixteen tokens, sixteen warps: a warp computes both gates of its token in one interleaved pass
    const int t = warp;
    if (t < T) {
      const int ei = (E + 31) >> 5;
      uint32_t allow[2] = {0u, 0u};
#pragma unroll 1
      for (int i = 0; i < ei; ++i) {
        const int e = lane + 32 * i;
        if (e < E) {
          allow[0] |= 1u << i;
          if (R->e2s[e] >= 0) allow[1] |= 1u << i;
        }
      }
      int se[2][kMaxTopK];
      float sg[2][kMaxTopK];
      dec_topk_gate2(slog + t * (kMaxE + 1), allow, ei, k, a.renorm, lane, se, sg);
      if (lane == 0) {
        const float xn = Q->xn[t];
#pragma unroll
        for (int j = 0; j < kMaxTopK; ++j) {
          if (j < k) {
            const int p = t * k + j;
            const size_t gp = (size_t)(tok0 + t) * k + j;
            const float gu = alive ? sg[0][j] : 0.f, gm = alive ? sg[1][j] : 0.f;
            const int sl = R->e2s[se[1][j]];
            Q->ue[p] = se[0][j];
            a.uidx[gp] = se[0][j]; a.ugate[gp] = gu;
            Q->pt[p] = xn * fabsf(gu) * Q->enorm[se[0][j]];
            Q->sl[p] = sl;
            a.midx[gp] = se[1][j]; a.mgate[gp] = gm; a.slot[gp] = sl;
            Q->pm[p] = xn * fabsf(gm) * Q->enorm[se[1][j]];
          }
        }
        a.xnorm[tok0 + t] = xn;
      }
    }
  } else {
  // gates: task = (token, pass); pass 0 the off-the-shelf gate, pass 1 the masked one; 2 TOK tasks over 16 warps
#pragma unroll 1
  for (int task = warp; task < 2 * TOK; task += kDecWarps) {
    const int t = task & (TOK - 1), pass = task / TOK;
    if (t >= T) continue;
    const int ei = (E + 31) >> 5;
    uint32_t allow = 0u;
#pragma unroll 1
    for (int i = 0; i < ei; ++i) {
      const int e = lane + 32 * i;
      if (e < E && (pass == 0 || R->e2s[e] >= 0)) allow |= 1u << i;
    }
    int se[kMaxTopK];
    float sg[kMaxTopK];
    dec_topk_gate(slog + t * (kMaxE + 1), allow, ei, k, a.renorm, lane, se, sg);
    if (lane == 0) {
      const float xn = Q->xn[t];
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j) {
        if (j < k) {
          const int p = t * k + j;
          const size_t gp = (size_t)(tok0 + t) * k + j;
          const float gv = alive ? sg[j] : 0.f;
          if (pass == 0) {
            Q->ue[p] = se[j];
            a.uidx[gp] = se[j]; a.ugate[gp] = gv;
            Q->pt[p] = xn * fabsf(gv) * Q->enorm[se[j]];
          } else {
            const int sl = R->e2s[se[j]];
            Q->sl[p] = sl;
            a.midx[gp] = se[j]; a.mgate[gp] = gv; a.slot[gp] = sl;
            Q->pm[p] = xn * fabsf(gv) * Q->enorm[se[j]];
          }
        }
      }
      if (pass == 0) a.xnorm[tok0 + t] = xn;
    }
  }
  }
  if (tid == 0) SWAPMOE_STAMP(0, 4);
#pragma unroll 1
  for (int i = tid; i < T * E; i += kDecThreads) {
    const int t = i / E, e = i - t * E;
    a.logits[(size_t)(tok0 + t) * E + e] = alive ? slog[t * (kMaxE + 1) + e] : 0.f;
  }
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 5);
  // per-CTA partial sums in pair order (at most 32 pairs): fixed order, run to run
  if (tid < E) {
    float s = 0.f;
    int n = 0;
#pragma unroll 8
    for (int p = 0; p < P; ++p)
      if (Q->ue[p] == tid) { s += Q->pt[p]; ++n; }
    a.cta_imp[(size_t)blockIdx.x * E + tid] = s;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + tid] = (float)n;
  }
  if (tid >= kDecThreads - K) {
    const int sl = kDecThreads - 1 - tid;                   // the last K threads: slot sums
    int c = 0;
    float m = 0.f;
#pragma unroll 8
    for (int p = 0; p < P; ++p)
      if (Q->sl[p] == sl) { ++c; m += Q->pm[p]; }
    a.cta_hist[(size_t)blockIdx.x * K + sl] = c;
    if (a.cta_mimp) a.cta_mimp[(size_t)blockIdx.x * K + sl] = m;
  }
  if (!alive && tid == 0) {
    // a wait gave up: let copies that may still be in flight land before the buffers are reused
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  if (tid == 0) SWAPMOE_STAMP(0, 6);
  finish_router_cta(a.scan, ring, 2 * kDecHalfBytes);       // the wave buffers are free: stage the scan inputs there
  if (tid == 0) SWAPMOE_STAMP(0, 10);
}

}  // namespace swapmoe
