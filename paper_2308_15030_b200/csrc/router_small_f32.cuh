// fp32 form of the small-batch router (SwapMoE Section 2 (G(x)), Fig. 4 (Masked Gating), Eq. 1
// (importance terms)): eight tokens per CTA, rows of x and of the router matrix as fp32 in shared
// memory, the product as split-TF32 warp-level mma (three m16n8k8 products per fp32 product, see
// gemm_tf32x3_kernel) with the contraction split over 16 warps.  Everything after the product is
// the bf16 kernel's.  The general fp32 router walks the contraction in 24-96 block-wide chunks with
// two barriers each (cfg1: 8 CTAs, 28 us); here all rows arrive with one memory latency.
#pragma once
#include "common.cuh"
#include "decode_fused.cuh"
#include "permute.cuh"
#include "router_args.cuh"
#include "router_small.cuh"
#include "gemm_mma.cuh"

namespace swapmoe {

// rows of an fp32 row-contiguous matrix (row length d) per wave: a power of two, at most 32
__host__ __device__ inline int rsf_rows_per_wave(int d) {
  int rp = 32;
  while (rp > 1 && rp * (d * 4 + kDecRowPad) > kDecHalfBytes) rp >>= 1;
  return rp;
}
__host__ __device__ inline RsSmem router_small_f32_layout(int d) {
  RsSmem m;
  int o = 2 * kDecHalfBytes;
  m.xs = o;    o += kRsTok * (d * 4 + kDecRowPad);
  m.slog = o;  o += kRsTok * (kMaxE + 1) * 4;
  o = (o + 15) & ~15;
  m.red = o;   o += kDecWarps * 32 * 8 * 4;
  m.route = o; o += (int)sizeof(DecRoute);
  o = (o + 15) & ~15;
  m.bars = o;  o += 16;
  m.pairs = o; o += (int)sizeof(RsRoute);
  m.total = o;
  return m;
}
inline size_t router_small_f32_smem_bytes(int d) { return (size_t)router_small_f32_layout(d).total + 1024; }

// dst[n * dst_stride + r] = <row r of the wave buffer, token n> for r < rows <= 32, n < n_tok <= 8 (fp32 rows,
// split-TF32 products; the contraction is split over the warps in steps of 8 and added in warp order).
__device__ __forceinline__ void rsf_wave_dots(const unsigned char* st, int rows, int d, const unsigned char* xs,
                                              int n_tok, float* red, float* dst, int dst_stride) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int pitch = d * 4 + kDecRowPad;
  float acc[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[i][q] = 0.f;
  // (row indices beyond what a wave buffer holds at this row length - 16 rows at d_model 768, 8 at 2048 - are clamped
  // to its last row: their products are dropped, and no read leaves the buffer)
  const int rmax = rsf_rows_per_wave(d) - 1;
  const float* ar[2][2];                                     // rows 16 i + 8 h + g of the buffer
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h) ar[i][h] = reinterpret_cast<const float*>(st + min(16 * i + 8 * h + g, rmax) * pitch) + t;
  const float* xrow = reinterpret_cast<const float*>(xs + min(g, n_tok - 1) * pitch) + t;
#pragma unroll 2
  for (int ks = warp; ks < d / 8; ks += kDecWarps) {
    const int k0 = ks * 8;
    uint32_t bh[2], bl[2];
    split_tf32(xrow[k0], bh[0], bl[0]);
    split_tf32(xrow[k0 + 4], bh[1], bl[1]);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      uint32_t ah[4], al[4];
      split_tf32(ar[i][0][k0], ah[0], al[0]);
      split_tf32(ar[i][1][k0], ah[1], al[1]);
      split_tf32(ar[i][0][k0 + 4], ah[2], al[2]);
      split_tf32(ar[i][1][k0 + 4], ah[3], al[3]);
      mma_tf32_16x8x8(acc[i], al, bh);
      mma_tf32_16x8x8(acc[i], ah, bl);
      mma_tf32_16x8x8(acc[i], ah, bh);
    }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float* rp = red + (warp * 32 + i * 16 + g) * 8 + 2 * t;
    *reinterpret_cast<float2*>(rp) = make_float2(acc[i][0], acc[i][1]);
    *reinterpret_cast<float2*>(rp + 8 * 8) = make_float2(acc[i][2], acc[i][3]);
  }
  __syncthreads();
  if (tid < 32 * 8) {
    const int r = tid >> 3, n = tid & 7;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) s += red[(w * 32 + r) * 8 + n];
    if (r < rows && n < n_tok) dst[n * dst_stride + r] = s;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kDecThreads, 1) router_small_f32_kernel(const RouterArgs a, int32_t* status) {
  constexpr int TOK = kRsTok;                               // tokens per CTA
  if ((int)blockIdx.x >= a.scan.n_cta) {                    // blocks beyond the token tiles prefetch weights
    pdl_wait();
    pdl_trigger();
    router_prefetch_role(a, a.scan.n_cta);
    return;
  }
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int d = a.d, E = a.E, k = a.k, K = a.K;
  const int chunks = d / 4, pitch = d * 4 + kDecRowPad;
  const RsSmem lay = router_small_f32_layout(d);
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
  const float* x = static_cast<const float*>(a.x) + (size_t)tok0 * d;
  const float* Wr = static_cast<const float*>(a.Wr);

  const int RW = rsf_rows_per_wave(d);
  const int n_rw = (E + RW - 1) / RW;
  auto issue_router_wave = [&](int w) {                     // all of warp 0
    const int rows = min(RW, E - w * RW);
    uint64_t* bar = &bars[w & 1];
    if (lane == 0) ptx::mbar_expect_tx(bar, (uint32_t)(rows * d * 4));
    __syncwarp();
    if (lane < rows)
      ptx::bulk_load_1d(ring + (w & 1) * kDecHalfBytes + lane * pitch, Wr + ((size_t)w * RW + lane) * d, (uint32_t)(d * 4), bar);
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
      const float4 u = *reinterpret_cast<const float4*>(xs + warp * pitch + c * 16);
      ss = fmaf(u.x, u.x, ss); ss = fmaf(u.y, u.y, ss); ss = fmaf(u.z, u.z, ss); ss = fmaf(u.w, u.w, ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) Q->xn[warp] = sqrtf(ss);
  }
  bool alive = true;
#pragma unroll 1
  for (int w = 0; w < n_rw; ++w) {
    if (!dec_wait_wave(bars, w, R, status, 25)) { alive = false; break; }
    rsf_wave_dots(ring + (w & 1) * kDecHalfBytes, min(RW, E - w * RW), d, xs, T, red, slog + w * RW, kMaxE + 1);
    if (warp == 0 && w + 2 < n_rw) {
      ptx::fence_proxy_async();
      issue_router_wave(w + 2);
    }
  }
  if (!alive)
    for (int i = tid; i < TOK * (kMaxE + 1); i += kDecThreads) slog[i] = 0.f;
  __syncthreads();
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
      if (Q->ue[p] == tid) { s += Q->pt[p]; ++n; }
    a.cta_imp[(size_t)blockIdx.x * E + tid] = s;
    if (a.cta_cnt) a.cta_cnt[(size_t)blockIdx.x * E + tid] = (float)n;
  }
  if (tid >= kDecThreads - K) {
    const int sl = kDecThreads - 1 - tid;                   // the last K threads: slot sums
    int c = 0;
    float m = 0.f;
#pragma unroll 1
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
  finish_router_cta(a.scan, ring, 2 * kDecHalfBytes);       // the wave buffers are free: stage the scan inputs there
}

}  // namespace swapmoe
