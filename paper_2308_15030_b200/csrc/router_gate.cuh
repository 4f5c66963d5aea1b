// Router product on the CUDA cores (fp32 layers, layers whose shape the tensor-core router does
// not take, and externally supplied logits), followed by the shared gate epilogue
// (SwapMoE Section 2: G(x); Fig. 4: Masked Gating; Eq. 1: importance terms).
#pragma once
#include "common.cuh"
#include "gate_epilogue.cuh"
#include "gemm_mma.cuh"
#include "permute.cuh"
#include "router_args.cuh"

namespace swapmoe {

constexpr int kRouterDK = 32;  // contraction chunk staged in shared memory
constexpr int kRouterLD = kRouterDK + 4;   // row pitch of the staged chunks (words): conflict-free mma fragment loads

inline size_t router_stage_floats(int E) {
  // token chunk [kTokTile][LD], router chunk [E rounded up to 8][LD], logits [kTokTile][E+1] + 8 of slack
  return (size_t)kTokTile * kRouterLD + (size_t)((E + 7) / 8 * 8) * kRouterLD + (size_t)kTokTile * (E + 1) + 8;
}
inline size_t router_smem_bytes(int E) {
  return ((router_stage_floats(E) * sizeof(float) + 15) & ~(size_t)15) + gate_smem_bytes();
}

// One CTA = kTokTile tokens.  The product runs as split-TF32 mma (three TF32 products per fp32
// product, see gemm_tf32x3_kernel): warp w owns the 16 tokens of half w & 1 and the 8-expert
// tiles (w >> 1), (w >> 1) + 4, ... (at most EI of them; EI, the number of 32-expert groups, is a
// template parameter that sizes the accumulators).  The global loads of chunk c + 2 are issued
// while chunk c is multiplied.
template <typename T, int EI>
__global__ void __launch_bounds__(kGateThreads) router_gate_kernel(const RouterArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int E = a.E;
  const int E8 = (E + 7) & ~7;
  float* xs = reinterpret_cast<float*>(smem_raw);              // [kTokTile][LD]
  float* ws = xs + kTokTile * kRouterLD;                       // [E8][LD] (rows beyond E are never written: their
                                                               //  products land in columns nobody reads)
  float* slog = ws + E8 * kRouterLD;                           // [kTokTile][E+1]
  const int stage_bytes = (int)(((size_t)(kTokTile * kRouterLD + E8 * kRouterLD +
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
    const int g = lane >> 2, t4 = lane & 3;
    const int m0 = (warp & 1) * 16, ng = warp >> 1, NT = E8 >> 3;
    float acc[EI][4];
#pragma unroll
    for (int j = 0; j < EI; ++j)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[j][q] = 0.f;
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
      __syncthreads();                       // the previous chunk's products are done
      sumsq += xv[set][0] * xv[set][0] + xv[set][1] * xv[set][1] + xv[set][2] * xv[set][2] + xv[set][3] * xv[set][3];
      store4(xs + lrow * kRouterLD + lcol, xv[set]);
#pragma unroll
      for (int i = 0; i < EI; ++i) {
        const int v = tid + kGateThreads * i;
        if (v < n_wv) store4(ws + (v >> 3) * kRouterLD + (v & 7) * 4, wv[set][i]);
      }
      __syncthreads();
      if (next_c0 < a.d) load_chunk(next_c0, set);
      const float* As = xs + (m0 + g) * kRouterLD + t4;
#pragma unroll
      for (int k0 = 0; k0 < kRouterDK; k0 += 8) {
        uint32_t ah[4], al[4];
        split_tf32(As[k0], ah[0], al[0]);
        split_tf32(As[8 * kRouterLD + k0], ah[1], al[1]);
        split_tf32(As[k0 + 4], ah[2], al[2]);
        split_tf32(As[8 * kRouterLD + k0 + 4], ah[3], al[3]);
#pragma unroll
        for (int j = 0; j < EI; ++j) {
          const int nt = ng + 4 * j;
          if (nt < NT) {
            const float* Bs = ws + (nt * 8 + g) * kRouterLD + t4 + k0;
            uint32_t bh[2], bl[2];
            split_tf32(Bs[0], bh[0], bl[0]);
            split_tf32(Bs[4], bh[1], bl[1]);
            mma_tf32_16x8x8(acc[j], al, bh);
            mma_tf32_16x8x8(acc[j], ah, bl);
            mma_tf32_16x8x8(acc[j], ah, bh);
          }
        }
      }
    };
    // The tensor core adds into its fp32 accumulators with truncation, so a long chain of accumulating mma drifts
    // (d_model 4096: 1536 dependent adds, 8e-4 on logits of magnitude 25).  Every 512 contraction elements the
    // accumulators are therefore added to the logits tile in shared memory with ordinary fp32 adds (each element
    // has one owner thread) and cleared.
    // accumulator layout: [0], [1] -> token m0 + g, experts 8 nt + 2 t4, + 1; [2], [3] -> token m0 + g + 8
    auto flush = [&](bool first) {
#pragma unroll
      for (int j = 0; j < EI; ++j) {
        const int nt = ng + 4 * j;
        if (nt < NT) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int e = nt * 8 + 2 * t4 + (q & 1);
            if (e < E) {
              float* dst = &slog[(m0 + g + (q >> 1) * 8) * (E + 1) + e];
              *dst = first ? acc[j][q] : *dst + acc[j][q];
            }
            acc[j][q] = 0.f;
          }
        }
      }
    };
    load_chunk(0, 0);
    if (kRouterDK < a.d) load_chunk(kRouterDK, 1);
    constexpr int kFlushCols = 512;
    bool first = true;
    for (int c0 = 0; c0 < a.d; c0 += 2 * kRouterDK) {
      stage_and_multiply(0, c0 + 2 * kRouterDK);
      if (c0 + kRouterDK < a.d) stage_and_multiply(1, c0 + 3 * kRouterDK);
      if ((c0 + 2 * kRouterDK) % kFlushCols == 0 && c0 + 2 * kRouterDK < a.d) { flush(first); first = false; }
    }
    flush(first);
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
