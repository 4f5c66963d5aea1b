// Grouped expert-FFN GEMM on the 5th-generation tensor cores (tcgen05 / TMEM / TMA),
// bf16 operands, fp32 accumulation.  SwapMoE Section 2: E_i(x) = W_out * act(W_in * x),
// evaluated per Virtual-Expert slot segment of the permuted token matrix.
//
// One persistent CTA per SM walks a list of 128-row output tiles:
//   warp 0   : TMA producer  (cp.async.bulk.tensor 2D, 128-byte swizzle, mbarrier tx)
//   warp 1   : MMA issuer    (one thread, tcgen05.mma kind::f16, M=128, N=BN, K=16)
//   warp 2   : TMEM allocator
//   warps 4-7: epilogue      (tcgen05.ld -> activation -> global stores), overlapped with
//                             the next tile's MMAs through two TMEM accumulator buffers.
// No load uses cluster multicast.  Every mbarrier wait is bounded: on expiry the
// kernel records a status word, stops issuing work, drains and frees its TMEM.
#pragma once
#include <cuda.h>

#include <cstdlib>

#include "../../include/swapmoe.h"
#include "common.cuh"

namespace swapmoe {

constexpr int kTcBM = 128;   // rows per tile (TMEM lanes)
constexpr int kTcBK = 64;    // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kTcUmmaK = 16;
constexpr int kTcThreads = 256;
constexpr int kTcSmemBudget = 200 * 1024;

// Epilogues: ReLU -> bf16 h; silu(a)*b -> bf16 h; plain fp32 y; and, for top-1 layers, the
// scatter-combine fused in: out[token(row)] = gate(row) * acc, written once per row in bf16.
enum { kTcEpiReluBf16 = 0, kTcEpiSwigluBf16 = 1, kTcEpiF32 = 2, kTcEpiScatterBf16 = 3 };

struct TcGemmArgs {
  void* C;                  // [rows_pad, ldc]
  const TileDesc* tiles;
  const int32_t* n_tiles;   // number of row tiles (device)
  int32_t* status;          // [0] = error flag, [1] = code of the wait that gave up
  int32_t ldc;              // columns of C
  int32_t n_col_tiles;      // column tiles per row tile
  int32_t k_blocks;         // contraction length / 64
  int32_t b_rows_per_phys;  // rows of the flattened weight map per arena entry
  int32_t b_rows_gate;      // row offset of the second input matrix (SwiGLU), else 0
  int32_t a_box_bytes;      // bytes one activation TMA box delivers (box rows * 128): small batches
                            // load only the first 16/32/64 rows of the 128-row MMA tile, the rest
                            // of the tile is stale shared memory whose output rows are never stored
  int32_t row_group;        // row tiles per scheduling group (see decode_tile)
  const int32_t* row_pair;  // [rows_pad] pair index of each padded row (scatter epilogue)
  const float* gate;        // [T*k] masked gate values (scatter epilogue)
  int32_t top_k;
  int32_t early_b;          // 1: the tile list is final when the CTAs start (see the kernel): weights are requested early
};

// ----------------------------------------------------------------------------- PTX wrappers
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
// Untiled bulk copy global -> shared memory (both 16-byte aligned, size a multiple of 16 bytes).
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

}  // namespace ptx

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes, written by
// TMA with 128-byte swizzle; 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address
  d |= (uint64_t)(1024u >> 4) << 32;             // stride between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Bounded wait: polls the barrier, and every 256 polls checks a 2-second deadline.
// Returns false (after recording `code`) when the wait gave up or another role aborted.
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                             int32_t* status, int code, uint64_t limit_ns = 2000000000ull) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((spin & 255u) == 0) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        if (atomicCAS(status, 0, 1) == 0) status[1] = code;
        return false;
      }
    }
  }
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nobody will ever complete,
// with a short limit; the wait must give up, record `code` and let the kernel return normally.
__global__ void bounded_wait_selftest_kernel(int32_t* status, int code, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) bounded_wait(&bar, 0u, &abort_flag, status, code, limit_ns);
  __syncthreads();
}

// Work item t -> (row tile, column tile).  Row tiles vary fastest inside a group of `group` row
// tiles, column tiles next, groups last: the row tiles of a slot (which share weights) run side
// by side, and for large problems the activations of one group stay in L2 while its column
// tiles are walked (group >= n_row_tiles: one group).
__device__ __forceinline__ void decode_tile(int t, int n_row_tiles, int n_col_tiles, int group, int* rt, int* ct) {
  group = min(group, n_row_tiles);
  const int per_group = group * n_col_tiles;
  const int g = t / per_group;
  const int r0 = g * group;
  const int rows_here = min(group, n_row_tiles - r0);
  const int u = t - g * per_group;
  *ct = u / rows_here;
  *rt = r0 + (u - *ct * rows_here);
}

// ----------------------------------------------------------------------------- epilogue stores
// An epilogue thread owns one accumulator row (a TMEM lane), so storing from its own registers
// makes every store instruction of a warp touch 32 different rows, 16 bytes each: 32 memory
// transactions per instruction, which saturate the load/store path that the TMA writes and the
// tensor core's operand reads also go through (measured on the 8192-token configuration: the
// mainloop slows down 3.5x while such an epilogue runs).  Instead each warp transposes 128 bytes
// per row through a private 4 KB staging buffer: the owner writes its row as eight 16-byte pieces,
// piece j at offset row * 128 + ((j ^ (row & 7)) * 16) (no bank conflicts), then lane l stores piece
// l & 7 of rows 4 i + (l >> 3), i = 0..7: a store instruction covers four rows of 128 contiguous
// bytes.
constexpr int kTcEpiWarpStage = 32 * 128;                 // bytes per epilogue warp
constexpr int kTcEpiStageBytes = 4 * kTcEpiWarpStage;     // four epilogue warps

// Destination of the rows this lane stores: dst[i] = start of the tile's columns in the output row of
// local row 4 i + (lane >> 3), plus this lane's 16 bytes; nullptr when that row is not stored.
// `drow_own` = output row (of the matrix C) of the row this lane owns, or -1.
__device__ __forceinline__ void epi_row_pointers(unsigned char* (&dst)[8], int drow_own, int lane, void* C, size_t ldc,
                                                 size_t col0, int elem_bytes) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int drow = __shfl_sync(0xffffffffu, drow_own, 4 * i + (lane >> 3));
    dst[i] = drow < 0 ? nullptr
                      : static_cast<unsigned char*>(C) + ((size_t)drow * ldc + col0) * elem_bytes + (lane & 7) * 16;
  }
}
// Stores 128 bytes of each of the warp's 32 rows: `pc` = the owned row's eight pieces, `byte_off` = offset of
// this 128-byte chunk from the start of the tile's columns.
__device__ __forceinline__ void epi_store_chunk(unsigned char* stg, const uint4 (&pc)[8], int lane,
                                                unsigned char* const (&dst)[8], int byte_off) {
  __syncwarp();                                            // the previous chunk has been read out
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<uint4*>(stg + lane * 128 + ((j ^ (lane & 7)) << 4)) = pc[j];
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = 4 * i + (lane >> 3);
    const uint4 v = *reinterpret_cast<const uint4*>(stg + row * 128 + (((lane & 7) ^ (row & 7)) << 4));
    if (dst[i] != nullptr) *reinterpret_cast<uint4*>(dst[i] + byte_off) = v;
  }
}

// The accumulator columns [c0, c0 + 32) of this thread's TMEM lane -> activation -> four 16-byte pieces
// (bf16 outputs) or eight (fp32 output).  `gate_cols` = distance to the gate columns (SwiGLU).
template <int EPI>
__device__ __forceinline__ void epi_load_pieces(uint32_t taddr, int c0, int gate_cols, float gate, uint4* pc) {
  uint32_t v[32];
  ptx::tmem_ld32(taddr + (uint32_t)c0, v);
  if (EPI == kTcEpiSwigluBf16) {
    uint32_t g[32];
    ptx::tmem_ld32(taddr + (uint32_t)(c0 + gate_cols), g);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float x1 = __uint_as_float(v[i]);
      v[i] = __float_as_uint(x1 / (1.f + __expf(-x1)) * __uint_as_float(g[i]));
    }
  } else {
    ptx::tmem_ld_wait();
  }
  if (EPI == kTcEpiF32) {
#pragma unroll
    for (int i = 0; i < 8; ++i) pc[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float f[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        f[j] = __uint_as_float(v[8 * i + j]);
        if (EPI == kTcEpiReluBf16) f[j] = fmaxf(f[j], 0.f);
        if (EPI == kTcEpiScatterBf16) f[j] *= gate;
      }
      pc[i] = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                         pack_bf16x2(f[6], f[7]));
    }
  }
}

// One accumulator (kOutCols output columns of this thread's row) -> global memory, 128 bytes per row and chunk.
template <int EPI, int kOutCols>
__device__ __forceinline__ void epi_store_tile(uint32_t taddr, unsigned char* stg, int lane, float gate,
                                               unsigned char* const (&dst)[8]) {
  constexpr int kElem = (EPI == kTcEpiF32) ? 4 : 2;
  constexpr int kChunkCols = 128 / kElem;                  // 32 fp32 or 64 bf16 columns
  static_assert(kOutCols % kChunkCols == 0, "whole 128-byte chunks");
#pragma unroll 1
  for (int c0 = 0; c0 < kOutCols; c0 += kChunkCols) {
    uint4 pc[8];
    epi_load_pieces<EPI>(taddr, c0, kOutCols, gate, pc);
    if (EPI != kTcEpiF32) epi_load_pieces<EPI>(taddr, c0 + 32, kOutCols, gate, pc + 4);
    epi_store_chunk(stg, pc, lane, dst, c0 * kElem);
  }
}

// MT = row sub-tiles of 128 rows that one CTA multiplies against the same weight tile.
template <int BN, int MT = 1>
struct TcSmem {
  static constexpr int kABytes = MT * kTcBM * kTcBK * 2;
  static constexpr int kBBytes = BN * kTcBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = (kTcSmemBudget - 2048) / kStageBytes;
  // + alignment slack and barriers (1 KB each) + the epilogue warps' staging buffers
  static constexpr int kBytes = kStages * kStageBytes + 2048 + kTcEpiStageBytes;
};

// C tile [128*MT, BN (or BN/2 for SwiGLU)] = epi(A[row0:row0+128*MT, :] * B[brow:brow+BN, :]^T).
// With MT = 2 a slot's weight tile is loaded once for two 128-row sub-tiles (two TMEM
// accumulators), which halves the weight bytes the SM has to ingest for slots with more
// than 128 rows; a tile with <= 128 valid rows skips the second half entirely.
template <int BN, int EPI, int MT = 1>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const TcGemmArgs a) {
  using S = TcSmem<BN, MT>;
  constexpr int kAccBufs = (2 * MT * BN <= 512) ? 2 : 1;   // TMEM accumulator sets
  constexpr int kHalfBytes = kTcBM * kTcBK * 2;
  constexpr int kStages = S::kStages;
  constexpr int kNB = (EPI == kTcEpiSwigluBf16) ? 2 : 1;   // weight boxes per stage
  constexpr int kBoxRows = BN / kNB;
  constexpr int kOutCols = BN / kNB;                        // output columns per tile
  constexpr uint32_t kTmemCols = kAccBufs * MT * BN;
  constexpr uint32_t kIdesc = make_idesc_bf16(kTcBM, BN);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* sA = smem;                                   // [stages][128][64] bf16
  unsigned char* sB = smem + kStages * S::kABytes;            // [stages][BN][64] bf16
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * S::kStageBytes);
  uint64_t* full = bars;                    // [stages]
  uint64_t* empty = bars + kStages;         // [stages]
  uint64_t* acc_full = bars + 2 * kStages;  // [2]
  uint64_t* acc_empty = acc_full + 2;       // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned char* epi_stage = smem + kStages * S::kStageBytes + 1024;   // [4 warps][32 rows][128 bytes]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kTr = (EPI == kTcEpiReluBf16 || EPI == kTcEpiSwigluBf16) ? 2 : 3;   // trace id: GEMM-1 or GEMM-2
  (void)kTr;

  if (threadIdx.x == 0) {
    SWAPMOE_STAMP(kTr, 0);
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 128); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 2) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The weights are constants of the layer, and for GEMM-2 the tile list is complete long before its CTAs can
  // start (it is written before GEMM-1's wait returns, and GEMM-2's CTAs are scheduled after that).  So with
  // `early_b` the producer requests the weight boxes of its first stages BEFORE the dependent-launch wait; only
  // the activations (written by the kernel in front) have to wait.  GEMM-1 may be scheduled while the kernels
  // that write the tile list still run, so it asks for nothing early.
  const bool is_producer = warp == 0 && lane == 0;
  int pre = 0;                                   // stages whose weight boxes are already requested
  if (is_producer && a.early_b) {
    const int n_rt = __ldcg(a.n_tiles);
    if ((int)blockIdx.x < n_rt * a.n_col_tiles) {
      int rt, ct;
      decode_tile((int)blockIdx.x, n_rt, a.n_col_tiles, a.row_group, &rt, &ct);
      const int4 raw = __ldcg(reinterpret_cast<const int4*>(a.tiles + rt));
      const TileDesc td = *reinterpret_cast<const TileDesc*>(&raw);
      const int brow = td.phys * a.b_rows_per_phys + ct * kBoxRows;
      const int halves = (MT == 2 && td.rows > kTcBM) ? 2 : 1;
      pre = a.k_blocks < kStages ? a.k_blocks : kStages;
      for (int kb = 0; kb < pre; ++kb) {
        ptx::mbar_expect_tx(&full[kb], (uint32_t)(halves * a.a_box_bytes + S::kBBytes));
#pragma unroll
        for (int j = 0; j < kNB; ++j)
          ptx::tma_load_2d(sB + kb * S::kBBytes + j * kBoxRows * kTcBK * 2, &tmB, &full[kb], kb * kTcBK,
                           brow + j * a.b_rows_gate);
      }
    }
  }
  if (is_producer) SWAPMOE_STAMP(kTr, 1);
  pdl_wait();      // the activations come from the preceding kernel
  pdl_trigger();
  // Which tile comes first depends on the tile count, and its descriptor is a second load behind that one: the
  // producer's warp fetches the first 32 descriptors together with the count (one per lane; the list's allocation
  // holds at least 32) and picks the right one by shuffle, so the two round trips overlap.
  int4 first_raw = make_int4(0, 0, 0, 0);
  if (warp == 0) first_raw = __ldcg(reinterpret_cast<const int4*>(a.tiles + lane));
  const int n_row_tiles = *a.n_tiles;
  const int total = n_row_tiles * a.n_col_tiles;
  int first_rt = -1;
  if (warp == 0 && (int)blockIdx.x < total) {
    int rt0, ct0;
    decode_tile((int)blockIdx.x, n_row_tiles, a.n_col_tiles, a.row_group, &rt0, &ct0);
    first_rt = rt0;
    const int src = rt0 & 31;
    first_raw.x = __shfl_sync(0xffffffffu, first_raw.x, src);
    first_raw.y = __shfl_sync(0xffffffffu, first_raw.y, src);
    first_raw.z = __shfl_sync(0xffffffffu, first_raw.z, src);
    first_raw.w = __shfl_sync(0xffffffffu, first_raw.w, src);
  }

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      SWAPMOE_STAMP(kTr, 2);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        int rt, ct;
        decode_tile(t, n_row_tiles, a.n_col_tiles, a.row_group, &rt, &ct);
        const TileDesc td = (t == (int)blockIdx.x && rt == first_rt && rt < 32)
                                ? *reinterpret_cast<const TileDesc*>(&first_raw) : a.tiles[rt];
        const int brow = td.phys * a.b_rows_per_phys + ct * kBoxRows;
        const int halves = (MT == 2 && td.rows > kTcBM) ? 2 : 1;
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          const bool early = t == (int)blockIdx.x && kb < pre;   // armed and weights requested above
          if (!early) {
            ok = bounded_wait(&empty[stage], phase ^ 1u, abort_flag, a.status, 1);
            if (!ok) break;
            ptx::mbar_expect_tx(&full[stage], (uint32_t)(halves * a.a_box_bytes + S::kBBytes));
          }
          for (int hf = 0; hf < halves; ++hf)
            ptx::tma_load_2d(sA + stage * S::kABytes + hf * kHalfBytes, &tmA, &full[stage], kb * kTcBK,
                             td.row0 + hf * kTcBM);
          if (!early) {
#pragma unroll
            for (int j = 0; j < kNB; ++j)
              ptx::tma_load_2d(sB + stage * S::kBBytes + j * kBoxRows * kTcBK * 2, &tmB, &full[stage],
                               kb * kTcBK, brow + j * a.b_rows_gate);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      SWAPMOE_STAMP(kTr, 3);                  // last load requested
      if (!ok) {
        // Give copies that are still in flight time to land before shared memory is released.
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      bool first_full = true;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        int halves = 1;
        {
          int rt, ct_unused;
          decode_tile(t, n_row_tiles, a.n_col_tiles, a.row_group, &rt, &ct_unused);
          if (MT == 2) halves = a.tiles[rt].rows > kTcBM ? 2 : 1;
        }
        ok = bounded_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status, 2);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * MT * BN);
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          ok = bounded_wait(&full[stage], phase, abort_flag, a.status, 3);
          if (!ok) break;
          if (first_full) { SWAPMOE_STAMP(kTr, 4); first_full = false; }
          ptx::tc_fence_after();
          const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(sB + stage * S::kBBytes));
          for (int hf = 0; hf < halves; ++hf) {
            const uint64_t da = make_kmajor_sw128_desc(ptx::smem_u32(sA + stage * S::kABytes + hf * kHalfBytes));
#pragma unroll
            for (int k = 0; k < kTcBK / kTcUmmaK; ++k) {
              // advancing 16 elements along K inside the swizzled row = +32 bytes = +2 in the address field
              ptx::umma_bf16(tmem_d + (uint32_t)(hf * BN), da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kIdesc,
                             (kb > 0 || k > 0) ? 1u : 0u);
            }
          }
          ptx::umma_commit(&empty[stage]);   // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(&acc_full[acc]);    // accumulator complete
        if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
      }
      SWAPMOE_STAMP(kTr, 5);                  // last MMA issued
    }
  } else if (warp >= 4) {
    // -------------------------------------------------------------------- epilogue
    const int q = warp - 4;                    // TMEM lane quarter this warp may read
    const int r = q * 32 + lane;               // row of the tile owned by this thread
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
      int rt, ct;
      decode_tile(t, n_row_tiles, a.n_col_tiles, a.row_group, &rt, &ct);
      const TileDesc td = a.tiles[rt];
      const int halves = (MT == 2 && td.rows > kTcBM) ? 2 : 1;
      // where this thread's rows go (and, for the scatter epilogue, their gate values): two dependent
      // global loads, fetched while the tile's MMAs are still running
      int drow_h[MT];                            // output row of C, -1: not stored
      float gate_h[MT];
#pragma unroll
      for (int hf = 0; hf < MT; ++hf) {
        const int rr = r + hf * kTcBM;           // row inside the (up to 256-row) tile
        const bool valid = hf < halves && rr < td.rows;
        drow_h[hf] = valid ? td.row0 + rr : -1;
        gate_h[hf] = 1.f;
        if (EPI == kTcEpiScatterBf16 && valid) {
          const int p = a.row_pair[td.row0 + rr];
          gate_h[hf] = a.gate[p];
          drow_h[hf] = p / a.top_k;
        }
      }
      ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 4);
      if (!ok) break;
      ptx::tc_fence_after();
#pragma unroll
      for (int hf = 0; hf < MT; ++hf) {
        if (hf < halves) {
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)((acc * MT + hf) * BN);
          constexpr int kElem = (EPI == kTcEpiF32) ? 4 : 2;
          if constexpr ((kOutCols * kElem) % 128 == 0) {
            unsigned char* dst[8];
            epi_row_pointers(dst, drow_h[hf], lane, a.C, (size_t)a.ldc, (size_t)ct * kOutCols, kElem);
            epi_store_tile<EPI, kOutCols>(taddr, epi_stage + q * kTcEpiWarpStage, lane, gate_h[hf], dst);
          } else {
            // 64 bytes per row (the narrowest bf16 tiles): every thread stores its own row
            uint4 pc[4];
            epi_load_pieces<EPI>(taddr, 0, kOutCols, gate_h[hf], pc);
            if (drow_h[hf] >= 0) {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<bf16*>(a.C) + (size_t)drow_h[hf] * a.ldc +
                                                    (size_t)ct * kOutCols);
#pragma unroll
              for (int i = 0; i < 4; ++i) dst[i] = pc[i];
            }
          }
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&acc_empty[acc]);       // 128 arrivals hand the buffer back to the MMA warp
      if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
    }
    if (threadIdx.x == 128) SWAPMOE_STAMP(kTr, 6);   // this CTA's last epilogue done
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

// Column-tile widths the kernels are built for.  Narrow tiles exist for small batches
// (decode): with few row tiles, wide column tiles would leave most SMs without work.
constexpr int kBn1Options[3] = {256, 128, 64};
constexpr int kBn2Options[4] = {256, 128, 64, 32};

struct TcState {
  bool enabled;
  int sm_count;
  PFN_encodeTiled encode;
  CUtensorMap map_xp[4], map_h[4];    // activations [rows_pad, d] / [rows_pad, f]; box rows 128, 64, 32, 16
  CUtensorMap map_win[3];             // W_in flattened to 2D, one map per entry of kBn1Options
  CUtensorMap map_wout[4];            // W_out flattened to 2D, one map per entry of kBn2Options
  CUtensorMap map_wr;                 // router matrix [E, d], box 64 x Epad
  bool arena_bound;
  bool router_ok;                     // tensor-core router usable (bf16 layer)
  int only;                           // 0: both grouped GEMMs; 1 / 2: launch only GEMM-1 / GEMM-2 (measurement re-runs)
};

inline bool tc_supported(const swapmoe_config_t& c) {
  return c.dtype == SWAPMOE_BF16 && c.d_model % 128 == 0 && c.d_ff % 256 == 0;
}

// Row sub-tiles per CTA for a forward of T tokens: two when the average slot has well over
// 128 rows (weight tiles are then shared by two sub-tiles), one for small slots (nothing to
// share) and for very large ones (tensor-bound: keep the double-buffered accumulators).
inline int tc_row_subtiles(const swapmoe_config_t& c, int T, bool cta_pairs = false) {
  const long long rows_per_slot = (long long)T * c.top_k / c.K;
  // CTA pairs (tc_gemm_pair_kernel) keep two accumulator sets, so they take the very large slots
  if (cta_pairs && rows_per_slot >= 1024 && c.d_model % 256 == 0) return 2;
  return (rows_per_slot >= 160 && rows_per_slot < 1024 && c.d_model % 256 == 0) ? 2 : 1;
}
// Whether a forward with 256-row tiles runs on CTA pairs: slots of at least `min_rows` rows on average (a
// 256-row tile with <= 128 valid rows leaves one SM of the pair idle, so ragged small slots stay with one CTA per tile).
inline bool tc_use_pairs(const swapmoe_config_t& c, int T, int n_pairs, int min_rows) {
  return n_pairs > 0 && (long long)T * c.top_k / c.K >= min_rows && c.d_model % 256 == 0 && c.d_ff % 256 == 0;
}

// Automatic choice: tensor cores whenever the shape allows it.
inline bool tc_selected(int path, const swapmoe_config_t& c, int /*T*/) {
  if (path == 1) return false;
  return tc_supported(c);
}

inline bool tc_encode_2d(PFN_encodeTiled enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kTcBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// View of a row-major bf16 matrix with a box of box_cols x box_rows elements and the given swizzle.
inline bool tc_encode_2d_box(PFN_encodeTiled enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                             uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle swizzle) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int EPI, int MT = 1>
inline bool tc_set_smem_attr() {
  return cudaFuncSetAttribute(tc_gemm_kernel<BN, EPI, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TcSmem<BN, MT>::kBytes) == cudaSuccess;
}

inline int32_t tc_init(TcState& s, const swapmoe_config_t& c, void* xp, void* h, float* /*y*/, int rows_pad) {
  s.enabled = false;
  s.arena_bound = false;
  s.router_ok = false;
  s.only = 0;
  if (c.dtype != SWAPMOE_BF16) return SWAPMOE_OK;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SWAPMOE_ERR_CUDA;
  if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SWAPMOE_ERR_CUDA;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) !=
          cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
    return SWAPMOE_ERR_CUDA;
  s.encode = reinterpret_cast<PFN_encodeTiled>(fn);
  s.router_ok = true;
  if (!tc_supported(c)) return SWAPMOE_OK;
  for (int i = 0; i < 4; ++i) {
    if (!tc_encode_2d(s.encode, &s.map_xp[i], xp, (uint64_t)rows_pad, (uint64_t)c.d_model, (uint32_t)(kTcBM >> i)))
      return SWAPMOE_ERR_CUDA;
    if (!tc_encode_2d(s.encode, &s.map_h[i], h, (uint64_t)rows_pad, (uint64_t)c.d_ff, (uint32_t)(kTcBM >> i)))
      return SWAPMOE_ERR_CUDA;
  }
  bool ok = tc_set_smem_attr<256, kTcEpiReluBf16>() && tc_set_smem_attr<128, kTcEpiReluBf16>() &&
            tc_set_smem_attr<64, kTcEpiReluBf16>() && tc_set_smem_attr<256, kTcEpiSwigluBf16>() &&
            tc_set_smem_attr<128, kTcEpiSwigluBf16>() && tc_set_smem_attr<64, kTcEpiSwigluBf16>() &&
            tc_set_smem_attr<256, kTcEpiF32>() && tc_set_smem_attr<128, kTcEpiF32>() &&
            tc_set_smem_attr<64, kTcEpiF32>() && tc_set_smem_attr<32, kTcEpiF32>() &&
            tc_set_smem_attr<256, kTcEpiScatterBf16>() && tc_set_smem_attr<128, kTcEpiScatterBf16>() &&
            tc_set_smem_attr<64, kTcEpiScatterBf16>() && tc_set_smem_attr<32, kTcEpiScatterBf16>() &&
            tc_set_smem_attr<256, kTcEpiF32, 2>() && tc_set_smem_attr<256, kTcEpiScatterBf16, 2>();
  if (!ok) return SWAPMOE_ERR_CUDA;
  s.enabled = true;
  return SWAPMOE_OK;
}

inline int32_t tc_bind_arena(TcState& s, const swapmoe_config_t& c, const void* arena_in, const void* arena_out) {
  if (!s.enabled) return SWAPMOE_OK;
  const int P = c.K + c.spare_slots;
  const int nin = c.act == SWAPMOE_ACT_SWIGLU ? 2 : 1;
  for (int i = 0; i < 3; ++i)     // SwiGLU loads W1 and W3 as two boxes of half the tile width
    if (!tc_encode_2d(s.encode, &s.map_win[i], arena_in, (uint64_t)P * nin * c.d_ff, (uint64_t)c.d_model,
                      (uint32_t)(kBn1Options[i] / nin)))
      return SWAPMOE_ERR_CUDA;
  for (int i = 0; i < 4; ++i)
    if (!tc_encode_2d(s.encode, &s.map_wout[i], arena_out, (uint64_t)P * c.d_model, (uint64_t)c.d_ff,
                      (uint32_t)kBn2Options[i]))
      return SWAPMOE_ERR_CUDA;
  s.arena_bound = true;
  return SWAPMOE_OK;
}

// Launch helper: programmatic dependent launch lets the kernel's prologue overlap the tail of
// the kernel before it on the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Column-tile width (index into `options`) that minimises the bytes the busiest SM has to pull:
// (tiles per SM) x (k-blocks) x (activation box + weight box).  Wide tiles amortise the
// activation box, narrow ones give every SM work when there are few row tiles.
inline int tc_pick_bn(const int* options, int n_options, int n, long long row_tiles, int sm_count, int a_box_bytes,
                      int min_bn) {
  int pick = -1;
  long long best = 0;
  for (int i = 0; i < n_options; ++i) {
    if (n % options[i] || options[i] < min_bn) continue;
    const long long tiles = row_tiles * (n / options[i]);
    const long long per_sm = (tiles + sm_count - 1) / sm_count;
    const long long cost = per_sm * (a_box_bytes + (long long)options[i] * kTcBK * 2);
    if (pick < 0 || cost < best) { pick = i; best = cost; }
  }
  return pick;
}

typedef void (*TcGemmKernel)(const CUtensorMap, const CUtensorMap, const TcGemmArgs);

}  // namespace swapmoe
