// Grouped expert-FFN GEMM on CUDA cores (FFMA, fp32 accumulate).  This is the fp32
// layer's contraction (a tensor-core fp32 path would need split-TF32 to hold the
// 1e-4 output tolerance) and the small-shape path of the bf16 layer.
// SwapMoE Section 2: E_i(x) = W_out * act(W_in * x), evaluated per slot segment.
#pragma once
#include "common.cuh"

namespace swapmoe {

constexpr int kSimtBM = 64, kSimtBN = 64, kSimtBK = 16;

struct SimtGemmArgs {
  const void* A;          // [rows_pad, Kdim] activations (TA)
  const void* W;          // arena: entry stride `slot_stride` elements; matrix [N, Kdim] (TW)
  void* C;                // [rows_pad, N] (TC)
  const TileDesc* tiles;
  const int32_t* n_tiles;
  long long slot_stride;  // elements between arena entries
  long long gate_offset;  // elements from W1 to W3 inside an entry (SwiGLU only)
  int32_t N, Kdim;
};

enum { kEpiNone = 0, kEpiRelu = 1, kEpiSwiglu = 2 };

// C[tile rows, 64 cols] = epi(A[tile rows, :] * W[phys][n0:n0+64, :]^T); grid = (N/64, max tiles).
template <typename TA, typename TW, typename TC, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const SimtGemmArgs a) {
  pdl_wait();
  pdl_trigger();
  if ((int)blockIdx.y >= *a.n_tiles) return;
  const TileDesc td = a.tiles[blockIdx.y];
  constexpr int LD = kSimtBM + 4;
  __shared__ __align__(16) float As[kSimtBK][LD];
  __shared__ __align__(16) float Bs[kSimtBK][LD];
  __shared__ __align__(16) float Gs[EPI == kEpiSwiglu ? kSimtBK : 1][LD];

  const int tid = threadIdx.x;
  const int n0 = blockIdx.x * kSimtBN;
  const TA* A = static_cast<const TA*>(a.A) + (size_t)td.row0 * a.Kdim;
  const TW* W = static_cast<const TW*>(a.W) + (size_t)td.phys * a.slot_stride + (size_t)n0 * a.Kdim;
  const TW* G = W + a.gate_offset;

  const int lr = tid >> 2, lc = (tid & 3) * 4;   // staged element: row lr, k-columns lc..lc+3
  const int ty = tid >> 4, tx = tid & 15;        // micro-tile: rows 4ty.., cols 4tx..

  float acc[4][4], acg[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; acg[i][j] = 0.f; }

  for (int k0 = 0; k0 < a.Kdim; k0 += kSimtBK) {
    float av[4], bv[4], gv[4];
    load4(A + (size_t)lr * a.Kdim + k0 + lc, av);
    load4(W + (size_t)lr * a.Kdim + k0 + lc, bv);
    if (EPI == kEpiSwiglu) load4(G + (size_t)lr * a.Kdim + k0 + lc, gv);
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      As[lc + q][lr] = av[q];
      Bs[lc + q][lr] = bv[q];
      if (EPI == kEpiSwiglu) Gs[lc + q][lr] = gv[q];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSimtBK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float ar[4] = {a4.x, a4.y, a4.z, a4.w};
      const float br[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
      if (EPI == kEpiSwiglu) {
        const float4 g4 = *reinterpret_cast<const float4*>(&Gs[kk][tx * 4]);
        const float gr[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acg[i][j] = fmaf(ar[i], gr[j], acg[i][j]);
      }
    }
  }
  TC* C = static_cast<TC*>(a.C) + (size_t)td.row0 * a.N + n0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = acc[i][j];
      if (EPI == kEpiRelu) v = fmaxf(v, 0.f);
      if (EPI == kEpiSwiglu) v = v / (1.f + expf(-v)) * acg[i][j];
      o[j] = v;
    }
    store4(C + (size_t)(ty * 4 + i) * a.N + tx * 4, o);
  }
}

}  // namespace swapmoe
