// Grouped expert GEMM for fp32 layers on the tcgen05 tensor cores (SwapMoE Section 2: the experts'
// FFN restricted to the resident slots), with fp32-grade accuracy from three bf16 products.
//
// No tensor-core input type holds fp32's 24 mantissa bits, and a single reduced-precision product cannot hold the
// 1e-4 output tolerance over 768-3072-term dot products.  Every operand is therefore split as x = b1 + b2 + rest
// with b1 = bf16(x) (round to nearest), b2 = bf16(x - b1) (the subtraction is exact in fp32) and |rest| below
// 2^-17 |x|; the product is b2_a*b1_b + b1_a*b2_b + b1_a*b1_b, accumulated in fp32 in TMEM, and the dropped terms
// are below 2^-16 relative.  (A first version split into TF32 pieces, hi = x with 13 mantissa bits cleared and
// lo = x - hi: same accuracy, but a kind::tf32 MMA covers 8 contraction elements where a kind::f16 one covers 16,
// and a tcgen05.mma costs about 110 clocks however small it is - the kernel is paced by the NUMBER of MMAs.)
//
// TMA brings the fp32 operands (k-blocks of 32 columns = 128-byte swizzled rows) into a ring of stages.  Two
// groups of four converter warps take alternate k-blocks.  The A operand goes to TENSOR MEMORY: converter thread r
// owns row r, reads its 32 values and writes 16 packed b1 pairs and 16 packed b2 pairs into 32 columns of TMEM
// lane r (`tcgen05.st`), so the MMAs read only B from shared memory.  The B operand is rewritten IN PLACE: a
// 128-byte row of 32 fp32 becomes [32 x b1 | 32 x b2], which is exactly a swizzled K-major bf16 row of 64, so no
// second buffer is needed.  The converters fence and arrive on `conv_done`; one thread then issues the 6 MMAs of
// the k-block (2 steps of K = 16, three products each) and commits to the barriers that free the stage and the
// TMEM slot.  Roles (512 threads): warp 0 TMA producer, warp 1 MMA issuer, warp 2 TMEM allocation, warps 4-7
// epilogue (two accumulator sets, so it overlaps the next item's MMAs), warps 8-11 and 12-15 the converter groups.
// A work item is (row tile, column tile, contraction slice): GEMM-2 has few output tiles and a long contraction, so
// its slices go to separate copies of y that the combine kernel adds in order (deterministic).
#pragma once
#include "gemm_tc.cuh"

namespace swapmoe {

constexpr int kF32BK = 32;                          // fp32 elements per k-block = one 128-byte swizzled row
constexpr int kF32BN = 128;                         // accumulator columns per tile (plain form)
constexpr int kF32Threads = 512;
constexpr int kF32ABytes = kTcBM * kF32BK * 4;      // 16 KB: the operand that goes to tensor memory
constexpr int kF32ASlots = 4;                       // tensor-memory slots of converted A k-blocks
constexpr int kF32ASlotCols = kF32BK;               // 16 columns of b1 pairs + 16 of b2 pairs
// Plain form: A = 128 token rows of a slot tile, B = 128 weight rows; C tile = [128 tokens, 128 outputs].
constexpr int kF32BBytes = kF32BN * kF32BK * 4;     // 16 KB
constexpr int kF32StageBytes = kF32ABytes + kF32BBytes;
constexpr int kF32Stages = 6;
constexpr int kF32TmemCols = 512;                   // 2 x 128 accumulator columns + 4 x 32 of A, rounded up
constexpr int kF32SmemBytes = kF32Stages * kF32StageBytes + 2048 + kTcEpiStageBytes;
// Swapped form for small slots: the 128 rows of the MMA (and of tensor memory) are WEIGHT rows, the accumulator's
// columns are the tokens of a slot tile (kF32SwapTok of them): 24 KB per k-block, eight stages.
constexpr int kF32SwapTok = 64;                     // token rows per tile = accumulator columns
constexpr int kF32SwapBBytes = kF32SwapTok * kF32BK * 4;                 // 8 KB
constexpr int kF32SwapStageBytes = kF32ABytes + kF32SwapBBytes;          // 24 KB
constexpr int kF32SwapStages = 8;
constexpr int kF32SwapTmemCols = 256;               // 2 x 64 accumulator columns + 4 x 32 of A
constexpr int kF32SwapSmemBytes = kF32SwapStages * kF32SwapStageBytes + 2048 + kTcEpiStageBytes;
static_assert(kF32SmemBytes <= 227 * 1024 && kF32SwapSmemBytes <= 227 * 1024, "shared memory per CTA");
static_assert(2 * kF32BN + kF32ASlots * kF32ASlotCols <= kF32TmemCols, "tensor memory of the plain form");
static_assert(2 * kF32SwapTok + kF32ASlots * kF32ASlotCols <= kF32SwapTmemCols, "tensor memory of the swapped form");

// Epilogues of the fp32 path (values continue the bf16 kernels' enum)
enum { kTcEpiReluF32 = 4, kTcEpiSwigluF32 = 5 };

struct TcF32Args {
  void* C;                  // [n_split][rows_pad, ldc] fp32
  const TileDesc* tiles;    // 128-row tiles
  const int32_t* n_tiles;
  int32_t* status;
  long long split_stride;   // elements between the copies of C
  int32_t ldc, n_col_tiles, k_blocks, n_split;   // k_blocks per slice
  int32_t b_rows_per_phys, b_rows_gate;
  int32_t early_b;          // 1: the tile list is final when the CTAs start: weights are requested before the wait
};

namespace ptx {
// A operand from tensor memory (lanes = rows, each 32-bit column = two consecutive bf16 of the contraction), B from
// shared memory.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(tmem_d),
      "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 consecutive 32-bit columns of this thread's TMEM lane <- registers
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
}  // namespace ptx

// x0, x1 -> (b1 pair, b2 pair): b1 = bf16(x) (round to nearest), b2 = bf16(x - b1); element 0 in the low half.
__device__ __forceinline__ void split_bf16_pair(uint32_t x0, uint32_t x1, uint32_t* p1, uint32_t* p2) {
  const float f0 = __uint_as_float(x0), f1 = __uint_as_float(x1);
  const __nv_bfloat162 b1 = __floats2bfloat162_rn(f0, f1);
  const uint32_t u1 = *reinterpret_cast<const uint32_t*>(&b1);
  const float r0 = f0 - __uint_as_float(u1 << 16), r1 = f1 - __uint_as_float(u1 & 0xffff0000u);   // exact
  const __nv_bfloat162 b2 = __floats2bfloat162_rn(r0, r1);
  *p1 = u1;
  *p2 = *reinterpret_cast<const uint32_t*>(&b2);
}

// accumulator columns [c0, c0 + 32) of this thread's TMEM lane -> activation -> eight 16-byte pieces of fp32
template <int EPI>
__device__ __forceinline__ void epi_load_pieces_f32(uint32_t taddr, int c0, int gate_cols, uint4* pc) {
  uint32_t v[32];
  ptx::tmem_ld32(taddr + (uint32_t)c0, v);
  if (EPI == kTcEpiSwigluF32) {
    uint32_t g[32];
    ptx::tmem_ld32(taddr + (uint32_t)(c0 + gate_cols), g);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float x1 = __uint_as_float(v[i]);
      v[i] = __float_as_uint(x1 / (1.f + expf(-x1)) * __uint_as_float(g[i]));
    }
  } else {
    ptx::tmem_ld_wait();
    if (EPI == kTcEpiReluF32) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(fmaxf(__uint_as_float(v[i]), 0.f));
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) pc[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}

// kSwap = false: A (128 rows, split into tensor memory) = token rows of a slot tile, B (shared memory) = 128 weight
// rows; C tile = [128 tokens, 128 outputs].  kSwap = true (ReLU / plain epilogues): A = 128 weight rows, B = the
// kF32SwapTok token rows of a slot tile; the accumulator holds C^T, lane = output column, column = token.
template <int EPI, bool kSwap = false>
__global__ void __launch_bounds__(kF32Threads, 1)
tc_gemm_f32_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const TcF32Args a) {
  static_assert(!(kSwap && EPI == kTcEpiSwigluF32), "the swapped form has no SwiGLU epilogue");
  constexpr int kNB = (EPI == kTcEpiSwigluF32) ? 2 : 1;     // weight boxes per stage
  constexpr int kBoxRows = kF32BN / kNB;
  constexpr int kOutCols = kF32BN / kNB;
  constexpr int kNRows = kSwap ? kF32SwapTok : kF32BN;      // rows of the B operand = accumulator columns
  constexpr int kBBytesK = kNRows * kF32BK * 4;             // bytes of the B operand per k-block
  constexpr int kStages = kSwap ? kF32SwapStages : kF32Stages;
  constexpr int kStageBytes = kSwap ? kF32SwapStageBytes : kF32StageBytes;
  constexpr int kSlots = kF32ASlots;                        // ring of converted k-blocks (TMEM slots of A)
  constexpr int kAccStride = kNRows;                        // TMEM columns per accumulator set
  constexpr int kASlotBase = 2 * kNRows;                    // first TMEM column of the A slots
  constexpr int kASlotCols = kF32ASlotCols;
  constexpr uint32_t kTmemCols = kSwap ? kF32SwapTmemCols : kF32TmemCols;
  constexpr uint32_t kIdesc = make_idesc_bf16(kTcBM, kNRows);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char* raw = smem;                                         // [stages][A 16 KB | B 16 or 8 KB]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  uint64_t* full = bars;                          // [stages]   TMA -> converters
  uint64_t* empty = full + kStages;               // [stages]   MMA -> producer
  uint64_t* conv_done = empty + kStages;          // [slots]    converters -> MMA (128 arrivals)
  uint64_t* lo_empty = conv_done + kSlots;        // [slots]    MMA -> converters (the TMEM slot is free)
  uint64_t* acc_full = lo_empty + kSlots;         // [2]
  uint64_t* acc_empty = acc_full + 2;             // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned char* epi_stage = reinterpret_cast<unsigned char*>(bars) + 1024;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kTr = (EPI == kTcEpiF32) ? 3 : 2;           // trace builds: kernel id of the stamps
  constexpr int kTrKb = 8;                                  // the k-block whose conversion and MMAs are stamped

  if (threadIdx.x == 0) {
    SWAPMOE_STAMP(kTr, 0);
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int s = 0; s < kSlots; ++s) { ptx::mbar_init(&conv_done[s], 128); ptx::mbar_init(&lo_empty[s], 1); }
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

  // As in tc_gemm_kernel: with `early_b` (GEMM-2: the tile list is final long before its CTAs start) the producer
  // requests the weight boxes of its first stages before the dependent-launch wait; only the activations have to wait.
  int pre = 0;
  if (warp == 0 && lane == 0 && a.early_b) {
    const int n_rt = __ldcg(a.n_tiles);
    const int per = n_rt * a.n_col_tiles;
    if ((int)blockIdx.x < per * a.n_split) {
      const int z = (int)blockIdx.x / per, u = (int)blockIdx.x - z * per;
      const int ct = u / n_rt, rt = u - ct * n_rt;
      const int4 rawd = __ldcg(reinterpret_cast<const int4*>(a.tiles + rt));
      const TileDesc td = *reinterpret_cast<const TileDesc*>(&rawd);
      const int brow = td.phys * a.b_rows_per_phys + ct * kBoxRows;
      pre = a.k_blocks < kStages ? a.k_blocks : kStages;
      for (int kb = 0; kb < pre; ++kb) {
        ptx::mbar_expect_tx(&full[kb], (uint32_t)(kF32ABytes + kBBytesK));
        if (kSwap) {
          ptx::tma_load_2d(raw + kb * kStageBytes, &tmA, &full[kb], (z * a.k_blocks + kb) * kF32BK, brow);
        } else {
#pragma unroll
          for (int j = 0; j < kNB; ++j)
            ptx::tma_load_2d(raw + kb * kStageBytes + kF32ABytes + j * kBoxRows * kF32BK * 4, &tmB, &full[kb],
                             (z * a.k_blocks + kb) * kF32BK, brow + j * a.b_rows_gate);
        }
      }
    }
  }
  if (threadIdx.x == 0) SWAPMOE_STAMP(kTr, 1);
  pdl_wait();
  pdl_trigger();
  if (threadIdx.x == 0) SWAPMOE_STAMP(kTr, 2);
  const int n_row_tiles = *a.n_tiles;
  const int per_slice = n_row_tiles * a.n_col_tiles;
  const int total = per_slice * a.n_split;        // item = slice * per_slice + (col tile * n_row_tiles + row tile)

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        const int z = t / per_slice, u = t - z * per_slice;
        const int ct = u / n_row_tiles, rt = u - ct * n_row_tiles;
        const TileDesc td = a.tiles[rt];
        const int brow = td.phys * a.b_rows_per_phys + ct * kBoxRows;
        const int kb0 = z * a.k_blocks;
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          const bool early = t == (int)blockIdx.x && kb < pre;   // armed and weights requested above
          unsigned char* sA = raw + stage * kStageBytes;
          if (!early) {
            ok = bounded_wait(&empty[stage], phase ^ 1u, abort_flag, a.status, 31);
            if (!ok) break;
            ptx::mbar_expect_tx(&full[stage], (uint32_t)(kF32ABytes + kBBytesK));
          }
          if (kSwap) {
            // tokens are the B operand, weights the A operand (the one that may have been requested early)
            ptx::tma_load_2d(sA + kF32ABytes, &tmB, &full[stage], (kb0 + kb) * kF32BK, td.row0);
            if (!early) ptx::tma_load_2d(sA, &tmA, &full[stage], (kb0 + kb) * kF32BK, brow);
          } else {
            ptx::tma_load_2d(sA, &tmA, &full[stage], (kb0 + kb) * kF32BK, td.row0);
            if (!early) {
#pragma unroll
              for (int j = 0; j < kNB; ++j)
                ptx::tma_load_2d(sA + kF32ABytes + j * kBoxRows * kF32BK * 4, &tmB, &full[stage], (kb0 + kb) * kF32BK,
                                 brow + j * a.b_rows_gate);
            }
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        SWAPMOE_STAMP(kTr, 3);
      }
      if (!ok) {
        // Give copies that are still in flight time to land before shared memory is released.
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      int stage = 0, slot = 0, acc = 0;
      uint32_t slot_phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        ok = bounded_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status, 32);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * kAccStride);
        for (int kb = 0; kb < a.k_blocks; ++kb) {
          ok = bounded_wait(&conv_done[slot], slot_phase, abort_flag, a.status, 33);
          if (!ok) break;
          ptx::tc_fence_after();
          if (kb == kTrKb && t == (int)blockIdx.x) SWAPMOE_STAMP(kTr, 14);
          // B row = [b1 of the 32 elements | b2 of them]: 16 elements = 32 bytes = +2 in the address field;
          // A slot = [8 columns b1 (k 0-15) | 8 b1 (k 16-31) | 8 b2 | 8 b2]; small terms first
          const uint64_t db = make_kmajor_sw128_desc(ptx::smem_u32(raw + stage * kStageBytes + kF32ABytes));
          const uint32_t a1 = tmem_base + (uint32_t)(kASlotBase + slot * kASlotCols), a2 = a1 + 16;
          ptx::umma_bf16_ts(tmem_d, a2, db, kIdesc, kb > 0 ? 1u : 0u);
          ptx::umma_bf16_ts(tmem_d, a2 + 8, db + 2, kIdesc, 1u);
          ptx::umma_bf16_ts(tmem_d, a1, db + 4, kIdesc, 1u);
          ptx::umma_bf16_ts(tmem_d, a1 + 8, db + 6, kIdesc, 1u);
          ptx::umma_bf16_ts(tmem_d, a1, db, kIdesc, 1u);
          ptx::umma_bf16_ts(tmem_d, a1 + 8, db + 2, kIdesc, 1u);
          ptx::umma_commit(&empty[stage]);       // the raw stage may be refilled
          ptx::umma_commit(&lo_empty[slot]);     // the TMEM slot may be rewritten
          if (kb == kTrKb && t == (int)blockIdx.x) SWAPMOE_STAMP(kTr, 15);
          if (++stage == kStages) stage = 0;
          if (++slot == kSlots) { slot = 0; slot_phase ^= 1u; }
        }
        if (!ok) break;
        ptx::umma_commit(&acc_full[acc]);
        SWAPMOE_STAMP(kTr, 5);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp >= 8) {
    // ---------------------------------------------------------------------- converters
    // two groups of four warps: group g converts the k-blocks whose slot has parity g (every other one), so two
    // conversions are in flight; both groups walk all k-blocks to keep stage and phase counters in step
    const int grp = (warp - 8) >> 2;
    const int ctid = (threadIdx.x - 8 * 32) & 127;   // 0..127 inside the group = row = TMEM lane
    int stage = 0, slot = 0;
    uint32_t phase = 0, slot_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
      for (int kb = 0; kb < a.k_blocks; ++kb) {
        if ((slot & 1) != grp) {
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
          if (++slot == kSlots) { slot = 0; slot_phase ^= 1u; }
          continue;
        }
        const bool tr = ctid == 0 && kb == kTrKb && t == (int)blockIdx.x;   // kTrKb is even: group 0 converts it
        if (ctid == 0 && grp == 0 && kb == 0 && t == (int)blockIdx.x) SWAPMOE_STAMP(kTr, 7);
        ok = bounded_wait(&full[stage], phase, abort_flag, a.status, 34);
        if (ctid == 0 && grp == 0 && kb == 0 && t == (int)blockIdx.x) SWAPMOE_STAMP(kTr, 4);
        if (tr) SWAPMOE_STAMP(kTr, 8);
        if (ok) ok = bounded_wait(&lo_empty[slot], slot_phase ^ 1u, abort_flag, a.status, 35);
        if (!ok) break;
        ptx::tc_fence_after();
        if (tr) SWAPMOE_STAMP(kTr, 9);
        {
          // A: thread = row (= TMEM lane); 32 values -> 16 packed b1 columns and 16 packed b2 columns
          const unsigned char* arow = raw + stage * kStageBytes + ctid * 128;
          uint32_t hm[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(arow + ((j ^ (ctid & 7)) << 4));
            split_bf16_pair(x.x, x.y, &hm[2 * j], &hm[16 + 2 * j]);
            split_bf16_pair(x.z, x.w, &hm[2 * j + 1], &hm[16 + 2 * j + 1]);
          }
          const uint32_t ta = tmem_base + ((uint32_t)((ctid >> 5) * 32) << 16) + (uint32_t)(kASlotBase + slot * kASlotCols);
          ptx::tmem_st32(ta, hm);
        }
        if (tr) SWAPMOE_STAMP(kTr, 10);
        // B: the first kNRows threads own a row each and rewrite it in place as [b1 x 32 | b2 x 32] (logical
        // 16-byte piece c at physical piece c ^ (row & 7), as the swizzled K-major bf16 row wants it)
        if (ctid < kNRows) {
          unsigned char* brow = raw + stage * kStageBytes + kF32ABytes + ctid * 128;
          uint32_t p1[16], p2[16];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(brow + ((j ^ (ctid & 7)) << 4));
            split_bf16_pair(x.x, x.y, &p1[2 * j], &p2[2 * j]);
            split_bf16_pair(x.z, x.w, &p1[2 * j + 1], &p2[2 * j + 1]);
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            *reinterpret_cast<uint4*>(brow + ((c ^ (ctid & 7)) << 4)) =
                make_uint4(p1[4 * c], p1[4 * c + 1], p1[4 * c + 2], p1[4 * c + 3]);
            *reinterpret_cast<uint4*>(brow + (((4 + c) ^ (ctid & 7)) << 4)) =
                make_uint4(p2[4 * c], p2[4 * c + 1], p2[4 * c + 2], p2[4 * c + 3]);
          }
        }
        if (tr) SWAPMOE_STAMP(kTr, 11);
        ptx::tmem_st_wait();
        if (tr) SWAPMOE_STAMP(kTr, 12);
        ptx::tc_fence_before();
        ptx::fence_proxy_async();                // these writes are read by the tensor core (async proxy)
        ptx::mbar_arrive(&conv_done[slot]);
        if (tr) SWAPMOE_STAMP(kTr, 13);
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
        if (++slot == kSlots) { slot = 0; slot_phase ^= 1u; }
      }
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------------------------- epilogue
    const int q = warp - 4;
    const int r = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
      const int z = t / per_slice, u = t - z * per_slice;
      const int ct = u / n_row_tiles, rt = u - ct * n_row_tiles;
      const TileDesc td = a.tiles[rt];
      if constexpr (kSwap) {
        // lane r holds output column ct * 128 + r of every token of the tile: a warp's 32 lanes store 128
        // contiguous bytes of one token row per instruction
        float* crow = static_cast<float*>(a.C) + (size_t)z * a.split_stride + (size_t)td.row0 * a.ldc +
                      (size_t)ct * kF32BN + r;
        ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 36);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccStride);
#pragma unroll 1
        for (int c0 = 0; c0 < kNRows; c0 += 32) {
          uint32_t v[32];
          ptx::tmem_ld32(taddr + (uint32_t)c0, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float f = __uint_as_float(v[i]);
            if (EPI == kTcEpiReluF32) f = fmaxf(f, 0.f);
            if (c0 + i < td.rows) crow[(size_t)(c0 + i) * a.ldc] = f;
          }
        }
      } else {
      const int drow = r < td.rows ? td.row0 + r : -1;
      unsigned char* dst[8];
      epi_row_pointers(dst, drow, lane, static_cast<float*>(a.C) + (size_t)z * a.split_stride, (size_t)a.ldc,
                       (size_t)ct * kOutCols, 4);
      ok = bounded_wait(&acc_full[acc], acc_phase, abort_flag, a.status, 36);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kF32BN);
#pragma unroll 1
      for (int c0 = 0; c0 < kOutCols; c0 += 32) {
        uint4 pc[8];
        epi_load_pieces_f32<EPI>(taddr, c0, kOutCols, pc);
        epi_store_chunk(epi_stage + q * kTcEpiWarpStage, pc, lane, dst, c0 * 4);
      }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&acc_empty[acc]);
      if (r == 0) SWAPMOE_STAMP(kTr, 6);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- host side
struct TcF32State {
  bool enabled, arena_bound;
  int sm_count;
  CUtensorMap map_xp, map_h;          // activations, box 32 x 128
  CUtensorMap map_win, map_wout;      // weights flattened to 2D; box 32 x 128 (64 for SwiGLU's W1 / W3)
  CUtensorMap map_xp_tok, map_h_tok;  // activations, box 32 x kF32SwapTok (swapped form)
  bool swap_ok;                       // the swapped form is available (ReLU layers)
  int only;                           // 0: both grouped GEMMs; 1 / 2: launch only GEMM-1 / GEMM-2 (measurement re-runs)
};

// The driver's tensor-map encoder (nullptr when it cannot be had).
inline PFN_encodeTiled tc_get_encoder() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return reinterpret_cast<PFN_encodeTiled>(fn);
}

inline bool tc_f32_supported(const swapmoe_config_t& c) {
  return c.dtype == SWAPMOE_F32 && c.d_model % kF32BN == 0 && c.d_ff % kF32BN == 0;
}

inline bool tc_encode_2d_f32(PFN_encodeTiled enc, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                             uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 4};
  const cuuint32_t box[2] = {(cuuint32_t)kF32BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int32_t tc_f32_init(TcF32State& s, PFN_encodeTiled enc, const swapmoe_config_t& c, void* xp, void* h,
                           int rows_pad, int sm_count) {
  s.enabled = false;
  s.arena_bound = false;
  s.only = 0;
  s.sm_count = sm_count;
  if (!enc || !tc_f32_supported(c)) return SWAPMOE_OK;
  if (!tc_encode_2d_f32(enc, &s.map_xp, xp, (uint64_t)rows_pad, (uint64_t)c.d_model, kTcBM) ||
      !tc_encode_2d_f32(enc, &s.map_h, h, (uint64_t)rows_pad, (uint64_t)c.d_ff, kTcBM) ||
      !tc_encode_2d_f32(enc, &s.map_xp_tok, xp, (uint64_t)rows_pad, (uint64_t)c.d_model, kF32SwapTok) ||
      !tc_encode_2d_f32(enc, &s.map_h_tok, h, (uint64_t)rows_pad, (uint64_t)c.d_ff, kF32SwapTok))
    return SWAPMOE_ERR_CUDA;
  s.swap_ok = c.act == SWAPMOE_ACT_RELU;
  if (s.swap_ok &&
      (cudaFuncSetAttribute(tc_gemm_f32_kernel<kTcEpiReluF32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            kF32SwapSmemBytes) != cudaSuccess ||
       cudaFuncSetAttribute(tc_gemm_f32_kernel<kTcEpiF32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                            kF32SwapSmemBytes) != cudaSuccess))
    return SWAPMOE_ERR_CUDA;
  if (cudaFuncSetAttribute(tc_gemm_f32_kernel<kTcEpiReluF32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kF32SmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_f32_kernel<kTcEpiSwigluF32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kF32SmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_f32_kernel<kTcEpiF32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kF32SmemBytes) != cudaSuccess)
    return SWAPMOE_ERR_CUDA;
  s.enabled = true;
  return SWAPMOE_OK;
}

inline int32_t tc_f32_bind_arena(TcF32State& s, PFN_encodeTiled enc, const swapmoe_config_t& c, const void* arena_in,
                                 const void* arena_out) {
  if (!s.enabled) return SWAPMOE_OK;
  const int P = c.K + c.spare_slots;
  const int nin = c.act == SWAPMOE_ACT_SWIGLU ? 2 : 1;
  if (!tc_encode_2d_f32(enc, &s.map_win, arena_in, (uint64_t)P * nin * c.d_ff, (uint64_t)c.d_model,
                        (uint32_t)(kF32BN / nin)) ||
      !tc_encode_2d_f32(enc, &s.map_wout, arena_out, (uint64_t)P * c.d_model, (uint64_t)c.d_ff, (uint32_t)kF32BN))
    return SWAPMOE_ERR_CUDA;
  s.arena_bound = true;
  return SWAPMOE_OK;
}

// Both grouped GEMMs of an fp32 layer.  GEMM-2 writes `*y_split` partial copies of y (the combine kernel adds them).
inline int32_t tc_ffn_f32(TcF32State& s, const swapmoe_config_t& c, void* h, float* y, long long y_copy_stride,
                          int y_copies, const TileDesc* tiles, const int32_t* n_tiles, int max_tiles, int n_tokens,
                          int32_t* status, cudaStream_t st, bool pdl, int64_t* launches, int* y_split,
                          cudaEvent_t between = nullptr, bool swapped = false) {
  if (!s.enabled || !s.arena_bound) return SWAPMOE_ERR_NOT_READY;
  const bool swiglu = c.act == SWAPMOE_ACT_SWIGLU;
  if (swapped && (swiglu || !s.swap_ok)) return SWAPMOE_ERR_UNSUPPORTED;
  const int tile_rows = swapped ? kF32SwapTok : kTcBM;
  const int out1 = swiglu ? kF32BN / 2 : kF32BN;
  TcF32Args g1;
  g1.C = h; g1.tiles = tiles; g1.n_tiles = n_tiles; g1.status = status; g1.split_stride = 0;
  g1.ldc = c.d_ff; g1.n_col_tiles = c.d_ff / out1; g1.k_blocks = c.d_model / kF32BK; g1.n_split = 1;
  g1.b_rows_per_phys = swiglu ? 2 * c.d_ff : c.d_ff;
  g1.b_rows_gate = swiglu ? c.d_ff : 0;
  g1.early_b = 0;
  long long work = (long long)max_tiles * g1.n_col_tiles;
  int grid = work > s.sm_count ? s.sm_count : (int)work;
  // (swapped form: the weight map is the A operand's, the token map with kF32SwapTok-row boxes the B operand's)
  cudaError_t e = s.only == 2 ? cudaSuccess :
                  swapped ? launch_kernel(tc_gemm_f32_kernel<kTcEpiReluF32, true>, dim3(grid), dim3(kF32Threads),
                                          kF32SwapSmemBytes, st, pdl, s.map_win, s.map_xp_tok, g1)
                  : swiglu ? launch_kernel(tc_gemm_f32_kernel<kTcEpiSwigluF32>, dim3(grid), dim3(kF32Threads), kF32SmemBytes,
                                           st, pdl, s.map_xp, s.map_win, g1)
                           : launch_kernel(tc_gemm_f32_kernel<kTcEpiReluF32>, dim3(grid), dim3(kF32Threads), kF32SmemBytes,
                                           st, pdl, s.map_xp, s.map_win, g1);
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  if (s.only != 2) ++*launches;
  if (between) cudaEventRecord(between, st);

  // GEMM-2: few output tiles, long contraction: slice it until every SM has an item
  const long long pairs = (long long)n_tokens * c.top_k;
  const long long touched = pairs < c.K ? pairs : c.K;
  const long long by_rows = pairs / tile_rows + touched / 2;
  const long long row_tiles_est = touched > by_rows ? touched : by_rows;
  const int n_col2 = c.d_model / kF32BN;
  int split = 1;
  while (split * 2 <= y_copies && row_tiles_est * n_col2 * split < s.sm_count &&
         (c.d_ff / kF32BK) % (split * 2) == 0 && c.d_ff / kF32BK / (split * 2) >= 8)
    split *= 2;
  TcF32Args g2;
  g2.C = y; g2.tiles = tiles; g2.n_tiles = n_tiles; g2.status = status; g2.split_stride = y_copy_stride;
  g2.ldc = c.d_model; g2.n_col_tiles = n_col2; g2.k_blocks = c.d_ff / kF32BK / split; g2.n_split = split;
  g2.b_rows_per_phys = c.d_model; g2.b_rows_gate = 0;
  g2.early_b = 1;
  work = (long long)max_tiles * n_col2 * split;
  grid = work > s.sm_count ? s.sm_count : (int)work;
  *y_split = split;
  if (s.only == 1) return SWAPMOE_OK;
  e = swapped ? launch_kernel(tc_gemm_f32_kernel<kTcEpiF32, true>, dim3(grid), dim3(kF32Threads), kF32SwapSmemBytes, st,
                              pdl && between == nullptr, s.map_wout, s.map_h_tok, g2)
              : launch_kernel(tc_gemm_f32_kernel<kTcEpiF32>, dim3(grid), dim3(kF32Threads), kF32SmemBytes, st,
                              pdl && between == nullptr, s.map_h, s.map_wout, g2);
  if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
  ++*launches;
  *y_split = split;
  return SWAPMOE_OK;
}

}  // namespace swapmoe
