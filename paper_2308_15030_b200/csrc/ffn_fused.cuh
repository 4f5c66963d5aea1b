// Both grouped expert-FFN GEMMs in ONE persistent tcgen05 kernel (bf16).
// SwapMoE Section 2: E_i(x) = W_out * act(W_in * x) per Virtual-Expert slot segment.
//
// At a few tens of MB of weights per GEMM the fixed cost of a launch (launch latency, the
// ramp until the TMA pipeline is full, the tail while the last tiles drain) is as large as
// the streaming time itself, so the two GEMMs share one grid: every CTA walks the GEMM-1
// tiles (h = act(xp * W_in^T)) and then the GEMM-2 tiles (y = h * W_out^T) of a common,
// statically ordered list.  A GEMM-2 tile needs the h rows of its row tile, i.e. all GEMM-1
// column tiles of that row tile: the epilogue of each GEMM-1 tile bumps a per-row-tile
// counter in global memory (each of its 128 epilogue threads adds one, with release
// semantics, after its own stores) and the GEMM-2 producer waits (bounded) until the counter
// is complete.  The wait cannot deadlock: a CTA waits only while it holds no unfinished GEMM-1
// tile (all of its own come first in its list), and GEMM-1 tiles never wait.
//
// Roles, pipeline, descriptors and the bounded waits are those of tc_gemm_kernel.
#pragma once
#include "gemm_tc.cuh"

namespace swapmoe {

struct TcFfnArgs {
  void* h;                   // [rows_pad, d_ff] bf16
  void* C2;                  // y fp32 [rows_pad, d_model] or out bf16 [T, d_model] (scatter)
  const TileDesc* tiles;
  const int32_t* n_tiles;
  int32_t* done;             // [row tiles] GEMM-1 column tiles finished (zeroed by the router's scan)
  int32_t* status;
  const int32_t* row_pair;
  const float* gate;
  int32_t top_k;
  int32_t d_model, d_ff;
  int32_t n_col1, kb1, b_rows_per_phys1, b_rows_gate1;
  int32_t n_col2, kb2, b_rows_per_phys2;
};

constexpr int kFfnStageBytes = kTcBM * kTcBK * 2 + 256 * kTcBK * 2;   // A 16 KB + B 32 KB
constexpr int kFfnStages = 4;
constexpr int kFfnSmemBytes = kFfnStages * kFfnStageBytes + 2048;

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// EPI1: kTcEpiReluBf16 or kTcEpiSwigluBf16.  BN2: column tile of GEMM-2.  EPI2: kTcEpiF32 or kTcEpiScatterBf16.
template <int EPI1, int BN2, int EPI2>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_ffn_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW2,
              const TcFfnArgs a) {
  constexpr int kStages = kFfnStages;
  constexpr int kABytes = kTcBM * kTcBK * 2, kBBytes = 256 * kTcBK * 2;
  constexpr int kNB1 = (EPI1 == kTcEpiSwigluBf16) ? 2 : 1;
  constexpr int kBox1 = 256 / kNB1, kOut1 = 256 / kNB1;
  constexpr uint32_t kIdesc1 = make_idesc_bf16(kTcBM, 256), kIdesc2 = make_idesc_bf16(kTcBM, BN2);
  constexpr uint32_t kBytes1 = kABytes + 256 * kTcBK * 2, kBytes2 = kABytes + BN2 * kTcBK * 2;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* sA = smem;
  unsigned char* sB = smem + kStages * kABytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kFfnStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 128); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmX); ptx::prefetch_tmap(&tmW1); ptx::prefetch_tmap(&tmH); ptx::prefetch_tmap(&tmW2);
  }
  if (warp == 2) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();
  pdl_trigger();
  const int n_row_tiles = *a.n_tiles;
  const int total1 = n_row_tiles * a.n_col1;
  const int total = total1 + n_row_tiles * a.n_col2;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total && ok; u += gridDim.x) {
        const bool p2 = u >= total1;
        const int v = p2 ? u - total1 : u;
        const int ct = v / n_row_tiles, rt = v - ct * n_row_tiles;   // row tiles vary fastest
        const TileDesc td = a.tiles[rt];
        const int kb_n = p2 ? a.kb2 : a.kb1;
        const CUtensorMap* mA = p2 ? &tmH : &tmX;
        const CUtensorMap* mB = p2 ? &tmW2 : &tmW1;
        const int brow = p2 ? td.phys * a.b_rows_per_phys2 + ct * BN2 : td.phys * a.b_rows_per_phys1 + ct * kBox1;
        if (p2) {
          // wait until every column tile of this row tile's h has been written
          const uint64_t t0 = ptx::globaltimer_ns();
          uint32_t spin = 0;
          while (ld_acquire(a.done + rt) < a.n_col1 * 128) {   // 128 epilogue threads per column tile
            if ((++spin & 63u) == 0) {
              if (*abort_flag) { ok = false; break; }
              if (ptx::globaltimer_ns() - t0 > 2000000000ull) {
                *abort_flag = 1;
                if (atomicCAS(a.status, 0, 1) == 0) a.status[1] = 21;
                ok = false;
                break;
              }
            }
          }
          if (!ok) break;
          asm volatile("fence.proxy.async;" ::: "memory");   // h was written through the generic proxy
        }
        for (int kb = 0; kb < kb_n; ++kb) {
          ok = bounded_wait(&empty[stage], phase ^ 1u, abort_flag, a.status, 1);
          if (!ok) break;
          ptx::mbar_expect_tx(&full[stage], p2 ? kBytes2 : kBytes1);
          ptx::tma_load_2d(sA + stage * kABytes, mA, &full[stage], kb * kTcBK, td.row0);
          if (p2) {
            ptx::tma_load_2d(sB + stage * kBBytes, mB, &full[stage], kb * kTcBK, brow);
          } else {
#pragma unroll
            for (int j = 0; j < kNB1; ++j)
              ptx::tma_load_2d(sB + stage * kBBytes + j * kBox1 * kTcBK * 2, mB, &full[stage], kb * kTcBK,
                               brow + j * a.b_rows_gate1);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total && ok; u += gridDim.x) {
        const bool p2 = u >= total1;
        const int kb_n = p2 ? a.kb2 : a.kb1;
        const uint32_t idesc = p2 ? kIdesc2 : kIdesc1;
        ok = bounded_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status, 2);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * 256);
        for (int kb = 0; kb < kb_n; ++kb) {
          ok = bounded_wait(&full[stage], phase, abort_flag, a.status, 3);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint64_t da = make_kmajor_sw128_desc(ptx::smem_u32(sA + stage * kABytes));
          const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(sB + stage * kBBytes));
#pragma unroll
          for (int k = 0; k < kTcBK / kTcUmmaK; ++k)
            ptx::umma_bf16(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc,
                           (kb > 0 || k > 0) ? 1u : 0u);
          ptx::umma_commit(&empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(&acc_full[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 4) {
    // -------------------------------------------------------------------- epilogue
    const int q = warp - 4;
    const int r = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < total && ok; u += gridDim.x) {
      const bool p2 = u >= total1;
      const int v = p2 ? u - total1 : u;
      const int ct = v / n_row_tiles, rt = v - ct * n_row_tiles;
      const TileDesc td = a.tiles[rt];
      ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 4);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * 256);
      const bool row_ok = r < td.rows;
      if (!p2) {
        bf16* hrow = static_cast<bf16*>(a.h) + (size_t)(td.row0 + r) * a.d_ff + (size_t)ct * kOut1;
#pragma unroll 1
        for (int c0 = 0; c0 < kOut1; c0 += 32) {
          uint32_t w[32];
          ptx::tmem_ld32(taddr + (uint32_t)c0, w);
          if (EPI1 == kTcEpiSwigluBf16) {
            uint32_t g[32];
            ptx::tmem_ld32(taddr + (uint32_t)(c0 + kOut1), g);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float x1 = __uint_as_float(w[i]);
              w[i] = __float_as_uint(x1 / (1.f + __expf(-x1)) * __uint_as_float(g[i]));
            }
          } else {
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(fmaxf(__uint_as_float(w[i]), 0.f));
          }
          if (row_ok) {
            uint4* dst = reinterpret_cast<uint4*>(hrow + c0);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[i] = make_uint4(pack_bf16x2(__uint_as_float(w[8 * i]), __uint_as_float(w[8 * i + 1])),
                                  pack_bf16x2(__uint_as_float(w[8 * i + 2]), __uint_as_float(w[8 * i + 3])),
                                  pack_bf16x2(__uint_as_float(w[8 * i + 4]), __uint_as_float(w[8 * i + 5])),
                                  pack_bf16x2(__uint_as_float(w[8 * i + 6]), __uint_as_float(w[8 * i + 7])));
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&acc_empty[acc]);
        // publish: every epilogue thread counts itself in once its own h stores are ordered before
        // the increment (release); no thread waits for another one here
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.done + rt) : "memory");
      } else {
        size_t crow = (size_t)(td.row0 + r) * a.d_model + (size_t)ct * BN2;
        float gate = 1.f;
        if (EPI2 == kTcEpiScatterBf16 && row_ok) {
          const int p = a.row_pair[td.row0 + r];
          gate = a.gate[p];
          crow = (size_t)(p / a.top_k) * a.d_model + (size_t)ct * BN2;
        }
#pragma unroll 1
        for (int c0 = 0; c0 < BN2; c0 += 32) {
          uint32_t w[32];
          ptx::tmem_ld32(taddr + (uint32_t)c0, w);
          ptx::tmem_ld_wait();
          if (row_ok) {
            if (EPI2 == kTcEpiF32) {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(a.C2) + crow + c0);
#pragma unroll
              for (int i = 0; i < 8; ++i)
                dst[i] = make_float4(__uint_as_float(w[4 * i]), __uint_as_float(w[4 * i + 1]),
                                     __uint_as_float(w[4 * i + 2]), __uint_as_float(w[4 * i + 3]));
            } else {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<bf16*>(a.C2) + crow + c0);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                dst[i] = make_uint4(
                    pack_bf16x2(gate * __uint_as_float(w[8 * i]), gate * __uint_as_float(w[8 * i + 1])),
                    pack_bf16x2(gate * __uint_as_float(w[8 * i + 2]), gate * __uint_as_float(w[8 * i + 3])),
                    pack_bf16x2(gate * __uint_as_float(w[8 * i + 4]), gate * __uint_as_float(w[8 * i + 5])),
                    pack_bf16x2(gate * __uint_as_float(w[8 * i + 6]), gate * __uint_as_float(w[8 * i + 7])));
            }
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&acc_empty[acc]);
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

template <int EPI1, int BN2, int EPI2>
inline cudaError_t tc_ffn_launch_one(const TcState& s, const TcFfnArgs& a, int grid, cudaStream_t st, bool pdl) {
  static bool attr_done = false;
  if (!attr_done) {
    const cudaError_t e = cudaFuncSetAttribute(tc_ffn_kernel<EPI1, BN2, EPI2>,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize, kFfnSmemBytes);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  return launch_kernel(tc_ffn_kernel<EPI1, BN2, EPI2>, dim3(grid), dim3(kTcThreads), kFfnSmemBytes, st, pdl,
                       s.map_xp[0], s.map_win[0], s.map_h[0], s.map_wout[BN2 == 256 ? 0 : 1], a);
}

// One launch for both GEMMs.  *combined tells whether out was written (top_k == 1).
inline int32_t tc_ffn_fused(TcState& s, const swapmoe_config_t& c, void* h, float* y, void* out, const TileDesc* tiles,
                            const int32_t* n_tiles, int32_t* done, const int32_t* row_pair, const float* mgate,
                            int max_tiles, int32_t* status, cudaStream_t st, bool pdl, int64_t* launches,
                            bool* combined) {
  if (!s.enabled || !s.arena_bound) return SWAPMOE_ERR_NOT_READY;
  const int bn2 = (c.d_model % 256 == 0 && c.d_model >= 2048) ? 256 : 128;
  const bool swiglu = c.act == SWAPMOE_ACT_SWIGLU;
  const bool scatter = c.top_k == 1;
  TcFfnArgs a;
  a.h = h; a.C2 = scatter ? out : static_cast<void*>(y);
  a.tiles = tiles; a.n_tiles = n_tiles; a.done = done; a.status = status;
  a.row_pair = row_pair; a.gate = mgate; a.top_k = c.top_k;
  a.d_model = c.d_model; a.d_ff = c.d_ff;
  a.n_col1 = swiglu ? c.d_ff / 128 : c.d_ff / 256;
  a.kb1 = c.d_model / kTcBK;
  a.b_rows_per_phys1 = swiglu ? 2 * c.d_ff : c.d_ff;
  a.b_rows_gate1 = swiglu ? c.d_ff : 0;
  a.n_col2 = c.d_model / bn2;
  a.kb2 = c.d_ff / kTcBK;
  a.b_rows_per_phys2 = c.d_model;
  long long work = (long long)max_tiles * (a.n_col1 + a.n_col2);
  const int grid = work > s.sm_count ? s.sm_count : (int)work;
  cudaError_t e;
#define SWAPMOE_FFN_CASE(E1, B2, E2) e = tc_ffn_launch_one<E1, B2, E2>(s, a, grid, st, pdl)
  if (swiglu) {
    if (bn2 == 256) { if (scatter) SWAPMOE_FFN_CASE(kTcEpiSwigluBf16, 256, kTcEpiScatterBf16); else SWAPMOE_FFN_CASE(kTcEpiSwigluBf16, 256, kTcEpiF32); }
    else              { if (scatter) SWAPMOE_FFN_CASE(kTcEpiSwigluBf16, 128, kTcEpiScatterBf16); else SWAPMOE_FFN_CASE(kTcEpiSwigluBf16, 128, kTcEpiF32); }
  } else {
    if (bn2 == 256) { if (scatter) SWAPMOE_FFN_CASE(kTcEpiReluBf16, 256, kTcEpiScatterBf16); else SWAPMOE_FFN_CASE(kTcEpiReluBf16, 256, kTcEpiF32); }
    else              { if (scatter) SWAPMOE_FFN_CASE(kTcEpiReluBf16, 128, kTcEpiScatterBf16); else SWAPMOE_FFN_CASE(kTcEpiReluBf16, 128, kTcEpiF32); }
  }
#undef SWAPMOE_FFN_CASE
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  ++*launches;
  *combined = scatter;
  return SWAPMOE_OK;
}

}  // namespace swapmoe
