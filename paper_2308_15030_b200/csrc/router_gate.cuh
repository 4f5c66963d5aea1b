// Router product on the CUDA cores (fp32 layers, layers whose shape the tensor-core router does
// not take, and externally supplied logits), followed by the shared gate epilogue
// (SwapMoE Section 2: G(x); Fig. 4: Masked Gating; Eq. 1: importance terms).
#pragma once
#include "common.cuh"
#include "gate_epilogue.cuh"
#include "permute.cuh"
#include "router_args.cuh"

namespace swapmoe {

constexpr int kRouterDK = 32;  // contraction chunk staged in shared memory

inline size_t router_stage_floats(int E) {
  // token chunk [kTokTile][DK+1], router chunk [E][DK+1], logits [kTokTile][E+1] + 8 of slack
  return (size_t)kTokTile * (kRouterDK + 1) + (size_t)E * (kRouterDK + 1) + (size_t)kTokTile * (E + 1) + 8;
}
inline size_t router_smem_bytes(int E) {
  return ((router_stage_floats(E) * sizeof(float) + 15) & ~(size_t)15) + gate_smem_bytes();
}

// One CTA = kTokTile tokens.  In the product warp w owns tokens 4w..4w+3 and lane l owns
// experts l + 32 i, i < EI (EI, the number of 32-expert groups, is a template parameter so that
// a layer with few experts carries no dead multiply-adds); the next chunk's global loads are
// issued before the current chunk's multiply-adds so their latency hides behind the arithmetic.
template <typename T, int EI>
__global__ void __launch_bounds__(kGateThreads) router_gate_kernel(const RouterArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int E = a.E;
  float* xs = reinterpret_cast<float*>(smem_raw);              // [kTokTile][DK+1]
  float* ws = xs + kTokTile * (kRouterDK + 1);                 // [E][DK+1]
  float* slog = ws + E * (kRouterDK + 1);                      // [kTokTile][E+1]
  const int stage_bytes = (int)(((size_t)(kTokTile * (kRouterDK + 1) + E * (kRouterDK + 1) +
                                          kTokTile * (E + 1) + 8) * sizeof(float) + 15) & ~(size_t)15);
  const GateSmem g = gate_smem_carve(smem_raw + stage_bytes);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tok0 = blockIdx.x * kTokTile;
  const T* x = static_cast<const T*>(a.x);
  const T* Wr = static_cast<const T*>(a.Wr);
  const bool have_ext = a.ext_logits != nullptr;

  pdl_wait();
  pdl_trigger();
  gate_load_tables(a, g);

  const int lrow = tid >> 3;         // token row this thread stages (0..31); == warp*4 + lane/8
  const int lcol = (tid & 7) * 4;    // 4 consecutive contraction indices
  const int ltok = tok0 + lrow;
  const int n_wv = E * (kRouterDK / 4);   // 4-element loads per router chunk
  float sumsq = 0.f;

  if (have_ext) {
    // logits come from the caller; x is read only for ||x||
    for (int c0 = 0; c0 < a.d; c0 += kRouterDK) {
      float xv[4] = {0.f, 0.f, 0.f, 0.f};
      if (ltok < a.T) load4(x + (size_t)ltok * a.d + c0 + lcol, xv);
      sumsq += xv[0] * xv[0] + xv[1] * xv[1] + xv[2] * xv[2] + xv[3] * xv[3];
    }
    for (int i = tid; i < kTokTile * E; i += kGateThreads) {
      const int r = i / E, e = i - r * E;
      slog[r * (E + 1) + e] = (tok0 + r < a.T) ? a.ext_logits[(size_t)(tok0 + r) * E + e] : 0.f;
    }
  } else {
    float acc[4][EI];
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
      for (int i = 0; i < EI; ++i) acc[t][i] = 0.f;
    // two register sets: the global loads of chunk c + 2 are issued while chunk c is multiplied, so a
    // load has two chunk periods to land (one period is shorter than the memory latency)
    float xv[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    float wv[2][EI][4];
    auto load_chunk = [&](int c0, int set) {
      if (ltok < a.T) load4(x + (size_t)ltok * a.d + c0 + lcol, xv[set]);
#pragma unroll
      for (int i = 0; i < EI; ++i) {
        const int v = tid + kGateThreads * i;
        if (v < n_wv) load4(Wr + (size_t)(v >> 3) * a.d + c0 + (v & 7) * 4, wv[set][i]);
      }
    };
    auto stage_and_multiply = [&](int set, int next_c0) {
      __syncthreads();                       // the previous chunk's multiply-adds are done
      sumsq += xv[set][0] * xv[set][0] + xv[set][1] * xv[set][1] + xv[set][2] * xv[set][2] + xv[set][3] * xv[set][3];
#pragma unroll
      for (int q = 0; q < 4; ++q) xs[lrow * (kRouterDK + 1) + lcol + q] = xv[set][q];
#pragma unroll
      for (int i = 0; i < EI; ++i) {
        const int v = tid + kGateThreads * i;
        if (v < n_wv) {
#pragma unroll
          for (int q = 0; q < 4; ++q) ws[(v >> 3) * (kRouterDK + 1) + (v & 7) * 4 + q] = wv[set][i][q];
        }
      }
      __syncthreads();
      if (next_c0 < a.d) load_chunk(next_c0, set);
#pragma unroll 8
      for (int kk = 0; kk < kRouterDK; ++kk) {
        float xr[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) xr[t] = xs[(warp * 4 + t) * (kRouterDK + 1) + kk];
#pragma unroll
        for (int i = 0; i < EI; ++i) {
          const int e = lane + 32 * i;
          const float w = (e < E) ? ws[e * (kRouterDK + 1) + kk] : 0.f;
#pragma unroll
          for (int t = 0; t < 4; ++t) acc[t][i] = fmaf(xr[t], w, acc[t][i]);
        }
      }
    };
    load_chunk(0, 0);
    if (kRouterDK < a.d) load_chunk(kRouterDK, 1);
    for (int c0 = 0; c0 < a.d; c0 += 2 * kRouterDK) {
      stage_and_multiply(0, c0 + 2 * kRouterDK);
      if (c0 + kRouterDK < a.d) stage_and_multiply(1, c0 + 3 * kRouterDK);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
      for (int i = 0; i < EI; ++i) {
        const int e = lane + 32 * i;
        if (e < E) slog[(warp * 4 + t) * (E + 1) + e] = acc[t][i];
      }
  }
  // ||x||^2 of a row: 8 consecutive lanes hold its partial sums
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 1);
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 2);
  sumsq += __shfl_xor_sync(0xffffffffu, sumsq, 4);
  if ((tid & 7) == 0) g.snorm[lrow] = sqrtf(sumsq);
  __syncthreads();
  gate_epilogue(a, g, slog, kTokTile, tok0, false, smem_raw, stage_bytes);
}

typedef void (*RouterGateKernel)(const RouterArgs);

// The instantiation for a layer with E experts.
template <typename T>
inline RouterGateKernel router_gate_fn(int E) {
  if (E <= 32) return router_gate_kernel<T, 1>;
  if (E <= 64) return router_gate_kernel<T, 2>;
  if (E <= 128) return router_gate_kernel<T, 4>;
  return router_gate_kernel<T, 8>;
}

// Raises the dynamic shared-memory limit of every instantiation (once per device).
template <typename T>
inline cudaError_t router_gate_set_smem_limit() {
  const int bytes = (int)router_smem_bytes(kMaxE);
  cudaError_t e = cudaFuncSetAttribute(router_gate_kernel<T, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(router_gate_kernel<T, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(router_gate_kernel<T, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(router_gate_kernel<T, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  return e;
}

}  // namespace swapmoe
