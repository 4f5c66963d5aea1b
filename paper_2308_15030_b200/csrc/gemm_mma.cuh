// Grouped expert-FFN GEMM on warp-level tensor-core instructions at fp32 accuracy (mma.sync TF32,
// three products per fp32 product).  It serves the layers whose shapes the tcgen05 kernels do not
// take: fp32 layers with d_model or d_ff not a multiple of 128, bf16 layers with d_model not a
// multiple of 128 or d_ff not a multiple of 256, and any layer when the caller selects it
// (swapmoe_set_gemm_path).  SwapMoE Section 2: E_i(x) = W_out * act(W_in * x), per slot segment.
//
// One CTA (256 threads) = 64 rows x 64 columns of one slot segment.  Shared memory keeps both
// operands row-major with the contraction index contiguous, as they sit in global memory, so a
// chunk is staged with 16-byte stores; the contraction runs in chunks through two shared-memory
// buffers and two register sets: the global loads of chunk c + 2 are issued before the arithmetic
// of chunk c, and chunk c + 1 (in registers since the previous round) moves to the other buffer
// afterwards; one barrier per chunk.  gridDim.z > 1 splits the contraction: slice z writes its
// partial sums to C + z * split_stride and the consumer adds the slices in order (a fixed order,
// so results repeat run to run).
#pragma once
#include "common.cuh"

namespace swapmoe {

constexpr int kMmaBM = 64, kMmaBN = 64, kMmaBK = 16, kMmaThreads = 256;

struct MmaGemmArgs {
  const void* A;          // [rows_pad, Kdim] activations (TA)
  const void* W;          // arena: entry stride `slot_stride` elements; matrix [N, Kdim] (TW)
  void* C;                // [rows_pad, N] (TC); slice z of a split contraction at C + z * split_stride
  const TileDesc* tiles;
  const int32_t* n_tiles;
  long long slot_stride;  // elements between arena entries
  long long gate_offset;  // elements from W1 to W3 inside an entry (SwiGLU only)
  long long split_stride; // elements between the partial outputs of a split contraction
  int32_t N, Kdim;
};

enum { kEpiNone = 0, kEpiRelu = 1, kEpiSwiglu = 2 };

__device__ __forceinline__ void store1(float* p, float v) { *p = v; }
__device__ __forceinline__ void store1(bf16* p, float v) { *p = __float2bfloat16_rn(v); }

// The products run on the tensor cores at fp32 accuracy: every fp32 operand is
// split into hi (its upper 19 bits, exactly a TF32 number) and lo = x - hi (exact in fp32, below
// 2^-10 |x|), and a product is three TF32 mma: hi*hi + lo*hi + hi*lo (the dropped lo*lo term and
// the rounding of lo to TF32 are below 2^-20 relative).  Accumulation is fp32 in the mma.
// Warp w owns rows 16 (w & 3) .. +15 and columns
// 32 (w >> 2) .. +31 as four m16n8k8 tiles.  The shared-memory pitch of 20 words makes the
// fragment loads conflict-free.
__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}

template <typename TA, typename TW, typename TC, int EPI>
__global__ void __launch_bounds__(kMmaThreads, 2) gemm_tf32x3_kernel(const MmaGemmArgs a) {
  pdl_wait();
  pdl_trigger();
  if ((int)blockIdx.y >= *a.n_tiles) return;
  const TileDesc td = a.tiles[blockIdx.y];
  // chunks of 32 (whole 128-byte lines per request), of 16 where a third operand (SwiGLU's gate
  // matrix) shares the 48 KB of static shared memory
  constexpr int BK = EPI == kEpiSwiglu ? 16 : 32;
  constexpr int kVec = BK / 4;                 // 16-byte pieces per row and chunk
  constexpr int kRowsPerPass = kMmaThreads / kVec;
  constexpr int kPasses = kMmaBM / kRowsPerPass;
  constexpr int LD = BK + 4;
  constexpr bool kGate = EPI == kEpiSwiglu;
  constexpr int kOperands = kGate ? 3 : 2;
  __shared__ __align__(16) float smem[2 * kOperands * kMmaBM * LD];   // [buffer][operand A / W / gate][row][LD]
  auto tile = [&](int buf, int op) { return smem + (size_t)(buf * kOperands + op) * kMmaBM * LD; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * kMmaBN;
  const int k_len = a.Kdim / (int)gridDim.z, k_begin = (int)blockIdx.z * k_len;
  const TA* A = static_cast<const TA*>(a.A) + (size_t)td.row0 * a.Kdim + k_begin;
  const TW* W = static_cast<const TW*>(a.W) + (size_t)td.phys * a.slot_stride + (size_t)n0 * a.Kdim + k_begin;
  const TW* G = W + a.gate_offset;
  const int lr = tid / kVec, lc = (tid % kVec) * 4;   // staging: rows lr + passes, contraction columns lc..lc+3
  const int m0 = (warp & 3) * 16, nb0 = (warp >> 2) * 32;

  float acc[4][4], acg[kGate ? 4 : 1][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll
  for (int i = 0; i < (kGate ? 4 : 1); ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acg[i][j] = 0.f;

  float av[2][kPasses][4], bv[2][kPasses][4], gv[kGate ? 2 : 1][kPasses][4];   // two register sets
  auto load_chunk = [&](int k0, int set) {
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) {
      const int r = lr + ps * kRowsPerPass;
      load4(A + (size_t)r * a.Kdim + k0 + lc, av[set][ps]);
      load4(W + (size_t)r * a.Kdim + k0 + lc, bv[set][ps]);
      if (kGate) load4(G + (size_t)r * a.Kdim + k0 + lc, gv[kGate ? set : 0][ps]);
    }
  };
  auto store_chunk = [&](int buf, int set) {
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) {
      const int r = lr + ps * kRowsPerPass;
      store4(tile(buf, 0) + r * LD + lc, av[set][ps]);
      store4(tile(buf, 1) + r * LD + lc, bv[set][ps]);
      if (kGate) store4(tile(buf, kGate ? 2 : 0) + r * LD + lc, gv[kGate ? set : 0][ps]);
    }
  };
  auto compute_chunk = [&](int buf) {
    const float* As = tile(buf, 0) + (m0 + g) * LD + t;
    const float* Bs = tile(buf, 1) + (nb0 + g) * LD + t;
    const float* Gs = tile(buf, kGate ? 2 : 0) + (nb0 + g) * LD + t;
#pragma unroll
    for (int k0 = 0; k0 < BK; k0 += 8) {
      uint32_t ah[4], al[4];
      split_tf32(As[k0], ah[0], al[0]);
      split_tf32(As[8 * LD + k0], ah[1], al[1]);
      split_tf32(As[k0 + 4], ah[2], al[2]);
      split_tf32(As[8 * LD + k0 + 4], ah[3], al[3]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        uint32_t bh[2], bl[2];
        split_tf32(Bs[nt * 8 * LD + k0], bh[0], bl[0]);
        split_tf32(Bs[nt * 8 * LD + k0 + 4], bh[1], bl[1]);
        mma_tf32_16x8x8(acc[nt], al, bh);
        mma_tf32_16x8x8(acc[nt], ah, bl);
        mma_tf32_16x8x8(acc[nt], ah, bh);
        if (kGate) {
          split_tf32(Gs[nt * 8 * LD + k0], bh[0], bl[0]);
          split_tf32(Gs[nt * 8 * LD + k0 + 4], bh[1], bl[1]);
          mma_tf32_16x8x8(acg[kGate ? nt : 0], al, bh);
          mma_tf32_16x8x8(acg[kGate ? nt : 0], ah, bl);
          mma_tf32_16x8x8(acg[kGate ? nt : 0], ah, bh);
        }
      }
    }
  };
  const int n_chunks = k_len / BK;
  load_chunk(0, 0);
  store_chunk(0, 0);
  if (n_chunks > 1) load_chunk(BK, 1);
  __syncthreads();
  for (int c = 0; c < n_chunks; c += 2) {
    if (c + 2 < n_chunks) load_chunk((c + 2) * BK, 0);
    compute_chunk(0);
    if (c + 1 < n_chunks) store_chunk(1, 1);
    __syncthreads();
    if (c + 1 >= n_chunks) break;
    if (c + 3 < n_chunks) load_chunk((c + 3) * BK, 1);
    compute_chunk(1);
    if (c + 2 < n_chunks) store_chunk(0, 0);
    __syncthreads();
  }
  // accumulator layout of the mma: [0], [1] -> row g, columns 2t, 2t+1; [2], [3] -> row g + 8
  TC* C = static_cast<TC*>(a.C) + (size_t)blockIdx.z * a.split_stride + (size_t)(td.row0 + m0 + g) * a.N + n0 + nb0 + 2 * t;
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = acc[nt][j];
      if (EPI == kEpiRelu) v = fmaxf(v, 0.f);
      if (kGate) v = v / (1.f + expf(-v)) * acg[kGate ? nt : 0][j];
      store1(C + (size_t)(j >> 1) * 8 * a.N + nt * 8 + (j & 1), v);
    }
  }
}

// Number of contraction slices for a GEMM with `tiles` output tiles of the 64 x 64 shape: enough
// to give every SM about two CTAs, at most `max_split`, and only slicings that leave whole chunks.
inline int mma_pick_split(long long tiles, int sm_count, int Kdim, int max_split) {
  int split = 1;
  while (split * 2 <= max_split && tiles * split < 2ll * sm_count && Kdim % (split * 2 * 32) == 0 &&
         Kdim / (split * 2) >= 64)
    split *= 2;
  return split;
}

}  // namespace swapmoe
