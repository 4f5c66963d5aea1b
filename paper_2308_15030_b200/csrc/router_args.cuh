// Arguments of the router kernels (SwapMoE Section 2, Fig. 4, Eq. 1).
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

// Role of the blocks beyond the router's token tiles: pull the resident experts' matrices towards
// L2 (GEMM-1's first, in slot order) while the router leaves HBM idle.
__device__ __forceinline__ void router_prefetch_role(const RouterArgs& a, int n_router_ctas) {
  constexpr long long kChunk = 16384;
  // chunks are dealt round-robin over the prefetch blocks: an SM sustains only about 200 GB/s of
  // prefetch requests, so the budget must be spread over enough of them to drain while the router runs
  const long long n_blk = (long long)gridDim.x - n_router_ctas;
  const long long n_pf = n_blk * blockDim.x;
  const long long me = (long long)threadIdx.x * n_blk + (blockIdx.x - n_router_ctas);
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
}

}  // namespace swapmoe
