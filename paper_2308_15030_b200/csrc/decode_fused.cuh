// Whole MoE-layer forward for a handful of tokens (decoding) in ONE launch, bf16.
// SwapMoE Section 2 (gate G(x), experts E_i), Fig. 4 (Masked Gating), Eq. 1 (importance).
//
// At one to eight tokens per step the layer is a pair of matrix-vector products per routed
// expert: what matters is that all SMs stream the touched experts' matrices at once and that
// nothing waits on a kernel boundary.  Design:
//   * Every CTA routes all tokens itself (router product, both gates, slots, the slot-sorted
//     pair order).  The arithmetic is identical in every CTA, so all agree bit for bit, and no
//     grid-wide exchange is needed before the expert matrices can be addressed.  The last CTA
//     of the grid also reports the routing (logits, selections, gates, slots, counts,
//     permutation) and adds the importance terms to the accumulators.
//   * Work item = (touched slot, block of 32 hidden units).  A CTA reads the 32 rows of W_in
//     (contiguous), forms the 32 hidden activations of every token routed to the slot, and
//     multiplies them into the matching 32 columns of W_out: a partial output row per pair.
//   * Every matrix byte reaches the SM through two 64.5 KB shared-memory buffers filled by TMA,
//     one "wave" each: untiled bulk copies, one per row into a padded pitch, for the router and
//     W_in rows; a 2-D tensor map (64-byte swizzle) for the 64-byte-wide column slices of W_out.
//     While one wave is multiplied the next is in flight, and an item's W_in and W_out waves are
//     requested together.  The router matrix is requested before the kernel waits for its
//     predecessor, since no kernel of this library writes it.
//   * The products run on the tensor cores with warp-level mma (m16n8k16, bf16 in, fp32 out):
//     the eight columns of the instruction are the (up to eight) tokens.  A CTA has few warps and
//     every phase runs once, so what counts is the number of dependent instructions per warp;
//     register-level mma needs a fiftieth of the instructions of the FFMA form and, unlike the
//     tcgen05 path of the large-batch kernels, no TMEM hand-offs.  The padded pitches and the
//     swizzle make every fragment load conflict-free.
//   * Partial rows are added in a fixed order in two steps, each done by whichever CTA finishes
//     last (an atomic ticket; nobody waits): first the 16 items of a group, then all groups,
//     gate-weighted, into `out`.
#pragma once
#include "common.cuh"
#include "gemm_tc.cuh"

namespace swapmoe {

constexpr int kDecMaxTokens = 8;      // tokens per launch = columns of one mma
constexpr int kDecMaxPairs = kDecMaxTokens * kMaxTopK;
constexpr int kDecThreads = 512;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecJB = 32;            // hidden units per work item
constexpr int kDecGroup = 16;         // work items per first-step sum
constexpr int kDecRowPad = 16;        // bytes added to a row's pitch in shared memory
constexpr int kDecHalfBytes = 66048;  // one wave buffer (32 rows of 2064 bytes; a multiple of 512); there are two
constexpr int kDecRecent = 4;         // recently served experts remembered per layer
constexpr int kDecOutRows = 256;      // rows of W_out per TMA box
constexpr int kDecOutBoxes = 4;       // boxes per W_out wave: 1024 rows
constexpr int kDecHPitch = 40;        // bf16 elements between the activation rows of two pairs (80 bytes)

struct DecodeArgs {
  const bf16* x;             // [T, d]
  const bf16* Wr;            // [E, d]
  const float* ext_logits;   // [T, E] or nullptr
  const int32_t* e2s;        // [E]
  const int32_t* s2e;        // [K]
  const int32_t* phys;       // [K] arena entry of each slot
  const float* enorm;        // [E]
  const bf16* arena_in;      // entries of in_stride elements: W_in [f, d] (SwiGLU: W1 then W3)
  const bf16* arena_out;     // entries of out_stride elements: W_out [d, f]
  long long in_stride, out_stride;
  float* logits; int32_t* uidx; float* ugate; int32_t* midx; float* mgate; int32_t* slot; float* xnorm;
  int32_t* count; int32_t* offset; int32_t* perm; int32_t* inv;
  float* imp; float* cnt; float* mimp;
  float* ypart;              // [f / 32][P][d] partial output rows per work item
  float* gpart;              // [groups][P][d] partial output rows per group
  unsigned* tickets;         // [K * groups + 1], all zero between launches
  bf16* out;                 // [T, d]
  int32_t* status;           // device status words (bounded waits report here)
  unsigned long long* touched;   // [1] running total of slots that received at least one pair, or nullptr
  // Activation locality (Section 2.2: successive tokens use consistent experts): the experts this layer
  // served most recently, most recent first (-1: none).  While the CTAs route, the first pf_depth of them
  // that are still resident are pulled towards L2; the reporting CTA then updates the list.
  int32_t* recent;               // [kDecRecent]
  unsigned long long* pf_stats;  // [2]: touched slots whose expert had been prefetched, touched slots
  int32_t pf_depth;              // 0: no prefetch
  int32_t T, d, f, E, k, K, renorm, swiglu;
};

// floats of partial-row workspace: ypart + gpart
inline size_t decode_ws_floats(int d, int f, int top_k) {
  const size_t P = (size_t)kDecMaxTokens * top_k, n_jb = f / kDecJB, groups = (n_jb + kDecGroup - 1) / kDecGroup;
  return (n_jb + groups) * P * d;
}
inline size_t decode_ticket_count(int f, int K) {
  const size_t n_jb = f / kDecJB, groups = (n_jb + kDecGroup - 1) / kDecGroup;
  return (size_t)K * groups + 1;
}
// rows of a row-contiguous matrix (row length d) per wave: a power of two, at most 32
__host__ __device__ inline int decode_rows_per_wave(int d) {
  int rp = 32;
  while (rp > 1 && rp * (d * 2 + kDecRowPad) > kDecHalfBytes) rp >>= 1;
  return rp;
}

// Order-preserving integer key of a logit: a > b  <=>  key(a) > key(b), equal logits (-0 and +0 included) have
// equal keys, and no finite or infinite logit maps to 0, which stands for "nothing available".
__device__ __forceinline__ uint32_t gate_key(float x) {
  const uint32_t b = __float_as_uint(x + 0.f);              // -0 becomes +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float gate_key_value(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Top-k of one token's logits by a whole warp: row[e] is the logit of expert e (shared memory), lane l looks
// at experts l, l + 32, ... of the `ei` 32-expert groups that exist; allow bit i says whether expert l + 32 i
// may be chosen; ties go to the lowest expert index.  Gate values are the softmax over the allowed experts (or
// over the selection when renorm is set).  Every lane returns the same selection.  The loops over the groups
// are rolled on purpose: the work follows E (with eight unrolled groups a 64-expert layer spent three quarters
// of the gate's instructions, accurate exponentials included, on experts that do not exist: 1.7 us per call),
// and the code stays small (one instantiation per group count ran 4 us slower: instruction fetch).
__device__ __forceinline__ void dec_topk_gate(const float* row, uint32_t allow, int ei, int k, int renorm, int lane,
                                              int (&sel_e)[kMaxTopK], float (&sel_g)[kMaxTopK]) {
  float sel_v[kMaxTopK];
  uint32_t avail = allow;
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j) {
    sel_e[j] = 0; sel_g[j] = 0.f; sel_v[j] = 0.f;
    if (j < k) {
      // the lane's best available logit as an order-preserving integer key (0: none; the first of equals
      // wins locally), then two warp reductions: the largest key, and the lowest index that holds it
      uint32_t bk = 0u;
      int be = 0x7fffffff;
#pragma unroll 1
      for (int i = 0; i < ei; ++i) {
        if ((avail >> i) & 1u) {
          const uint32_t key = gate_key(row[lane + 32 * i]);
          if (key > bk) { bk = key; be = lane + 32 * i; }
        }
      }
      const uint32_t kmax = __reduce_max_sync(0xffffffffu, bk);
      be = __reduce_min_sync(0xffffffffu, bk == kmax ? be : 0x7fffffff);
      sel_e[j] = be; sel_v[j] = gate_key_value(kmax);
      if ((be & 31) == lane) avail &= ~(1u << (be >> 5));
    }
  }
  const float m = sel_v[0];
  float den = 0.f;
  if (renorm) {
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j)
      if (j < k) den += expf(sel_v[j] - m);
  } else {
#pragma unroll 1
    for (int i = 0; i < ei; ++i)
      if ((allow >> i) & 1u) den += expf(row[lane + 32 * i] - m);
    den = warp_sum(den);
  }
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j)
    if (j < k) sel_g[j] = expf(sel_v[j] - m) / den;
}

// The off-the-shelf gate (allow[0]) and the masked gate (allow[1]) of one token in one pass: the two selections
// are independent instruction streams that the scheduler interleaves, so a warp that owns both gates of a token
// needs little more time than for one (a gate is a chain of dependent shuffles and exponentials, not work).
__device__ __forceinline__ void dec_topk_gate2(const float* row, const uint32_t (&allow)[2], int ei, int k, int renorm,
                                               int lane, int (&sel_e)[2][kMaxTopK], float (&sel_g)[2][kMaxTopK]) {
  float sel_v[2][kMaxTopK];
  uint32_t avail[2] = {allow[0], allow[1]};
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j) {
#pragma unroll
    for (int p = 0; p < 2; ++p) { sel_e[p][j] = 0; sel_g[p][j] = 0.f; sel_v[p][j] = 0.f; }
    if (j < k) {
      uint32_t bk[2] = {0u, 0u};
      int be[2] = {0x7fffffff, 0x7fffffff};
#pragma unroll 1
      for (int i = 0; i < ei; ++i) {
        const uint32_t key = gate_key(row[lane + 32 * i]);
#pragma unroll
        for (int p = 0; p < 2; ++p)
          if (((avail[p] >> i) & 1u) && key > bk[p]) { bk[p] = key; be[p] = lane + 32 * i; }
      }
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const uint32_t kmax = __reduce_max_sync(0xffffffffu, bk[p]);
        be[p] = __reduce_min_sync(0xffffffffu, bk[p] == kmax ? be[p] : 0x7fffffff);
        sel_e[p][j] = be[p]; sel_v[p][j] = gate_key_value(kmax);
        if ((be[p] & 31) == lane) avail[p] &= ~(1u << (be[p] >> 5));
      }
    }
  }
  const float m[2] = {sel_v[0][0], sel_v[1][0]};
  float den[2] = {0.f, 0.f};
  if (renorm) {
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j)
      if (j < k) { den[0] += expf(sel_v[0][j] - m[0]); den[1] += expf(sel_v[1][j] - m[1]); }
  } else {
#pragma unroll 1
    for (int i = 0; i < ei; ++i) {
      const float x = row[lane + 32 * i];
#pragma unroll
      for (int p = 0; p < 2; ++p)
        if ((allow[p] >> i) & 1u) den[p] += expf(x - m[p]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      den[0] += __shfl_xor_sync(0xffffffffu, den[0], o);
      den[1] += __shfl_xor_sync(0xffffffffu, den[1], o);
    }
  }
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j)
    if (j < k) { sel_g[0][j] = expf(sel_v[0][j] - m[0]) / den[0]; sel_g[1][j] = expf(sel_v[1][j] - m[1]) / den[1]; }
}

// Routing state of the launch, identical in every CTA (shared memory).
struct DecRoute {
  int ue[kDecMaxPairs], me[kDecMaxPairs], sl[kDecMaxPairs];   // per pair p = t*k + j
  float ug[kDecMaxPairs], mg[kDecMaxPairs];
  int q[kDecMaxPairs];          // position of pair p in slot-sorted order
  int pair_at[kDecMaxPairs];    // inverse: pair at sorted position
  int tok_at[kDecMaxPairs];     // token of the pair at sorted position
  int touched[kDecMaxPairs];    // slots with pairs, ascending
  int tcount[kDecMaxPairs];     // ... their pair counts
  int toffset[kDecMaxPairs];    // ... and the position of their first pair in sorted order
  int n_touched;
  int phys[kMaxSlots];          // arena entry of each slot
  int e2s[kMaxE];               // expert -> slot
  float xn[kDecMaxTokens];
  int last;                     // ticket outcome broadcast
  int abort_flag;               // a bounded wait gave up
  int tok[kDecMaxTokens];       // token behind each of the eight mma columns
};

// Shared-memory carve-up (bytes from the 1024-aligned base); xs rows are padded like the wave rows.
struct DecSmem {
  int xs, slog, hraw, hraw3, hsb, red, route, bars, total;
};
__host__ __device__ inline DecSmem decode_smem_layout(int d) {
  DecSmem m;
  int o = 2 * kDecHalfBytes;
  m.xs = o;    o += kDecMaxTokens * (d * 2 + kDecRowPad);
  m.slog = o;  o += kDecMaxTokens * (kMaxE + 1) * 4;
  o = (o + 15) & ~15;
  m.hraw = o;  o += kDecMaxPairs * kDecJB * 4;            // W1 x (fp32), [pair][32]
  m.hraw3 = o; o += kDecMaxPairs * kDecJB * 4;            // W3 x
  m.hsb = o;   o += kDecMaxPairs * kDecHPitch * 2;        // activations, bf16, [pair][40]
  m.red = o;   o += kDecWarps * 32 * 8 * 4;               // per-warp partial products [warp][32 rows][8 columns]
  m.route = o; o += (int)sizeof(DecRoute);
  o = (o + 15) & ~15;
  m.bars = o;  o += 16;
  m.total = o;
  return m;
}
inline size_t decode_smem_bytes(int d) { return (size_t)decode_smem_layout(d).total + 1024; }

__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lds32(const unsigned char* p) { return *reinterpret_cast<const uint32_t*>(p); }

// Waits for wave w (buffer w & 1, its barrier's phase (w >> 1) & 1): thread 0 polls (bounded), the
// block barrier releases the others, and every thread then observes the completed phase itself.
// Returns false when a wait gave up.
__device__ __noinline__ bool dec_wait_wave(uint64_t* bars, int w, DecRoute* R, int32_t* status, int code) {
  uint64_t* bar = &bars[w & 1];
  const uint32_t parity = (uint32_t)(w >> 1) & 1u;
  if (threadIdx.x == 0) bounded_wait(bar, parity, &R->abort_flag, status, code);
  __syncthreads();
  if (R->abort_flag) return false;
  if (!ptx::mbar_try_wait(bar, parity)) bounded_wait(bar, parity, &R->abort_flag, status, code);
  return true;
}

// dst[n * dst_stride + r] = <row r of the wave buffer, token R->tok[n]> for r < rows <= 32,
// n < nn <= 8.  The contraction is split over the warps in steps of 16; a warp multiplies its
// steps for both 16-row tiles, the per-warp partial products meet in `red` and are added in warp
// order.  Rows of the buffer beyond `rows` hold stale data whose products are dropped; row indices beyond what
// a wave buffer holds at this row length (fewer than 32 rows from d_model 2048 on) are clamped to its last row,
// so that no read leaves the buffer.
__device__ __noinline__ void dec_wave_dots(const unsigned char* st, int rows, int d, const unsigned char* xs,
                                           const DecRoute* R, int nn, float* red, float* dst, int dst_stride,
                                           int rows_held) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int pitch = d * 2 + kDecRowPad;
  float acc[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const unsigned char* xrow = xs + R->tok[g] * pitch + t * 4;
  const int rmax = rows_held - 1;              // rows_held = decode_rows_per_wave(d): what a wave buffer holds
  const unsigned char* ar[2][2];               // rows 16 i + 8 h + g of the buffer
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h) ar[i][h] = st + min(16 * i + 8 * h + g, rmax) * pitch + t * 4;
#pragma unroll 2
  for (int ks = warp; ks < d / 16; ks += kDecWarps) {
    const int kb = ks * 32;                    // byte offset of the step inside a row
    const uint32_t b0 = lds32(xrow + kb), b1 = lds32(xrow + kb + 16);
#pragma unroll
    for (int i = 0; i < 2; ++i)
      mma_bf16_16x8x16(acc[i], lds32(ar[i][0] + kb), lds32(ar[i][1] + kb), lds32(ar[i][0] + kb + 16),
                       lds32(ar[i][1] + kb + 16), b0, b1);
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
    if (r < rows && n < nn) dst[n * dst_stride + r] = s;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kDecThreads, 1)
decode_fused_kernel(const __grid_constant__ CUtensorMap tmWo, const DecodeArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~static_cast<uintptr_t>(1023));
  const int T = a.T, d = a.d, f = a.f, E = a.E, k = a.k, K = a.K;
  const int P = T * k, chunks = d / 8, pitch = d * 2 + kDecRowPad;
  const DecSmem lay = decode_smem_layout(d);
  unsigned char* ring = smem;                                  // two wave buffers
  unsigned char* xs = smem + lay.xs;                           // [8][pitch] token rows, bf16
  float* slog = reinterpret_cast<float*>(smem + lay.slog);     // [8][kMaxE + 1]
  float* hraw = reinterpret_cast<float*>(smem + lay.hraw);     // [pairs][32] W1 x
  float* hraw3 = reinterpret_cast<float*>(smem + lay.hraw3);   // [pairs][32] W3 x (SwiGLU)
  bf16* hsb = reinterpret_cast<bf16*>(smem + lay.hsb);         // [pairs][40] activations
  float* red = reinterpret_cast<float*>(smem + lay.red);
  DecRoute* R = reinterpret_cast<DecRoute*>(smem + lay.route);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + lay.bars);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const int RW = decode_rows_per_wave(d);            // rows of Wr / W_in per wave
  const bool have_ext = a.ext_logits != nullptr;
  const int n_rw = have_ext ? 0 : (E + RW - 1) / RW; // router waves
  // Rows of a row-major matrix -> padded rows of buffer (w & 1): lane r of warp 0 copies row r.
  auto issue_rows = [&](int w, const bf16* src, int rows) {
    uint64_t* bar = &bars[w & 1];
    if (lane == 0) ptx::mbar_expect_tx(bar, (uint32_t)(rows * d * 2));
    __syncwarp();
    if (lane < rows)
      ptx::bulk_load_1d(ring + (w & 1) * kDecHalfBytes + lane * pitch, src + (size_t)lane * d, (uint32_t)(d * 2), bar);
  };

  if (tid == 0) {
    ptx::mbar_init(&bars[0], 1);
    ptx::mbar_init(&bars[1], 1);
    R->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmWo);
    SWAPMOE_STAMP(0, 0);
  }
  __syncthreads();
  // the router matrix is a constant of the layer: request it before waiting for the predecessor
  if (warp == 0) {
    if (n_rw > 0) issue_rows(0, a.Wr, min(RW, E));
    if (n_rw > 1) issue_rows(1, a.Wr + (size_t)RW * d, min(RW, E - RW));
  }
  // The list of recently served experts was written by this layer's previous forward, which is long complete
  // (every kernel of the stream waits for the one in front of it): it may be read before the wait.
  int recent_e = -1;
  if (warp == kDecWarps - 1 && lane < a.pf_depth) recent_e = __ldcg(a.recent + lane);
  pdl_wait();
  pdl_trigger();
  if (tid == 0) SWAPMOE_STAMP(0, 1);
  // ------------------------------------------------------------------ routing, in every CTA
  // (integer divisions are kept out of this kernel's once-run paths: each costs dozens of
  // dependent instructions)
  // token t is copied by warps t and t + 8 (T <= 8, 16 warps), four independent loads per lane and round
  {
    const int t = warp & (kDecMaxTokens - 1);
    if (t < T) {
#pragma unroll 1
      for (int c0 = (warp >> 3) * 32 + lane; c0 < chunks; c0 += 256) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 64 * u < chunks) v[u] = reinterpret_cast<const uint4*>(a.x)[t * chunks + c0 + 64 * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c0 + 64 * u < chunks) *reinterpret_cast<uint4*>(xs + t * pitch + (c0 + 64 * u) * 16) = v[u];
      }
    }
  }
  if (tid < kMaxE) R->e2s[tid] = tid < E ? a.e2s[tid] : -1;
  if (tid < K) R->phys[tid] = a.phys[tid];
  if (tid < kDecMaxTokens) R->tok[tid] = min(tid, T - 1);
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 2);
  if (warp == kDecWarps - 1 && a.pf_depth > 0) {
    // L2 prefetch of the recently served experts that are resident: 16 KB chunks of both matrices, dealt over
    // the CTAs (chunk c of a slot goes to CTA c mod grid), so every SM issues a handful of requests
    constexpr int kChunk = 16384;
    const int n_in = (int)(a.in_stride * 2 / kChunk), n_out = (int)(a.out_stride * 2 / kChunk);
#pragma unroll 1
    for (int h = 0; h < a.pf_depth; ++h) {
      const int e = __shfl_sync(0xffffffffu, recent_e, h);
      const int sl = (e >= 0 && e < E) ? R->e2s[e] : -1;
      if (sl < 0) continue;
      const int ph = R->phys[sl];
      for (int c = (int)blockIdx.x + (int)gridDim.x * lane; c < n_in + n_out; c += (int)gridDim.x * 32) {
        const char* src = c < n_in
            ? reinterpret_cast<const char*>(a.arena_in + (size_t)ph * a.in_stride) + (size_t)c * kChunk
            : reinterpret_cast<const char*>(a.arena_out + (size_t)ph * a.out_stride) + (size_t)(c - n_in) * kChunk;
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"((unsigned)kChunk) : "memory");
      }
    }
  }
  if (warp < T && blockIdx.x == gridDim.x - 1) {     // ||x_t||: only the reporting CTA needs it
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
    if (lane == 0) R->xn[warp] = sqrtf(ss);
  }
  if (have_ext) {
#pragma unroll 1
    for (int i = tid; i < T * E; i += kDecThreads) {
      const int t = i / E, e = i - t * E;
      slog[t * (kMaxE + 1) + e] = a.ext_logits[i];
    }
  }
  bool alive = true;
#pragma unroll 1
  for (int w = 0; w < n_rw; ++w) {
    // router wave w holds rows w*RW .. of Wr
    if (!dec_wait_wave(bars, w, R, a.status, 21)) { alive = false; break; }
    dec_wave_dots(ring + (w & 1) * kDecHalfBytes, min(RW, E - w * RW), d, xs, R, T, red, slog + w * RW, kMaxE + 1, RW);
    if (warp == 0 && w + 2 < n_rw) {               // dec_wave_dots ends with a block barrier: the buffer is free
      ptx::fence_proxy_async();
      issue_rows(w + 2, a.Wr + (size_t)(w + 2) * RW * d, min(RW, E - (w + 2) * RW));
    }
  }
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 3);
  if (alive && warp < 2 * kDecMaxTokens && (warp & (kDecMaxTokens - 1)) < T) {
    // gate of token (warp & 7) (Section 2; Fig. 4): warps 0-7 the off-the-shelf gate, 8-15 the masked one
    const int t = warp & (kDecMaxTokens - 1), pass = warp / kDecMaxTokens;
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
#pragma unroll
      for (int j = 0; j < kMaxTopK; ++j) {
        if (j < k) {
          const int p = t * k + j;
          if (pass == 0) { R->ue[p] = se[j]; R->ug[p] = sg[j]; }
          else { R->me[p] = se[j]; R->mg[p] = sg[j]; R->sl[p] = R->e2s[se[j]]; }
        }
      }
    }
  }
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 4);
  // slot-sorted pair order (a stable counting sort on the flat pair index), by one warp: lane p
  // holds pair p; its position is (#pairs in lower slots) + (#earlier pairs in its own slot)
  if (warp == 0) {
    const int my = lane < P ? R->sl[lane] : 0x7fffffff;
    const unsigned peers = __match_any_sync(0xffffffffu, my);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int less = 0, leaders_less = 0;
#pragma unroll 1
    for (int p = 0; p < P; ++p) {
      const int o = __shfl_sync(0xffffffffu, my, p);
      const unsigned op = __shfl_sync(0xffffffffu, peers, p);
      const bool first = (op & ((1u << p) - 1u)) == 0u;      // pair p is the first of its slot
      less += (o < my);
      leaders_less += (first && o < my);
    }
    const unsigned leaders = __ballot_sync(0xffffffffu, lane < P && rank == 0);
    if (lane < P) {
      const int q = less + rank;
      R->q[lane] = q;
      R->pair_at[q] = lane;
      R->tok_at[q] = lane / k;
      if (rank == 0) {
        R->touched[leaders_less] = my;
        R->tcount[leaders_less] = __popc(peers);
        R->toffset[leaders_less] = less;
      }
    }
    if (lane == 0) R->n_touched = alive ? __popc(leaders) : 0;
  }
  __syncthreads();
  if (tid == 0) SWAPMOE_STAMP(0, 5);

  // -------------------------------------------------------------------- expert work items
  // Waves of an item, in the order they are requested and consumed: the 32 rows of W_in in
  // groups of RW rows (for SwiGLU: W1's groups, then W3's), then W_out's column slice in groups
  // of 1024 rows (four boxes).  Wave v of this CTA's sequence is wave n_rw + v overall.
  const int n_jb = f / kDecJB, n_groups = (n_jb + kDecGroup - 1) / kDecGroup;
  const int n_items = R->n_touched * n_jb;
  const int n_in = kDecJB / RW, n_mats = a.swiglu ? 2 : 1;
  const int out_rows = kDecOutRows * kDecOutBoxes;   // 1024
  const int n_out = (d + out_rows - 1) / out_rows;
  const int wpi = n_in * n_mats + n_out;             // waves per item
  // A CTA takes a contiguous range of items: consecutive items are consecutive blocks of hidden
  // units of one slot, so their partial output rows can be added in registers (a "run") and only
  // one set of partial rows, one fence and one ticket are spent per run instead of per item.
  const int ipc = (n_items + (int)gridDim.x - 1) / (int)gridDim.x;      // items per CTA
  const int item0 = (int)blockIdx.x * ipc;
  const int my_items = max(0, min(ipc, n_items - item0));
  const int total = my_items * wpi;
  // issue cursor of warp 0 (waves are requested strictly in order): wave, its index inside the
  // item, the item's slot index and hidden block
  int iv = 0, iwi = 0, iti = n_items > 0 ? item0 / n_jb : 0, ijb = n_items > 0 ? item0 - iti * n_jb : 0;
  auto issue_item_wave = [&]() {                     // all of warp 0; requests wave iv and advances
    const int wi = iwi, ti = iti, jb = ijb;
    const int ph = R->phys[R->touched[ti]];
    const int w = n_rw + iv;
    ++iv;
    if (++iwi == wpi) { iwi = 0; if (++ijb == n_jb) { ijb = 0; ++iti; } }
    if (wi < n_in * n_mats) {
      const int mat = wi >= n_in ? 1 : 0, rp = wi - mat * n_in;
      issue_rows(w, a.arena_in + (size_t)ph * a.in_stride + (size_t)mat * f * d + (size_t)(jb * kDecJB + rp * RW) * d, RW);
    } else {
      const int ow = wi - n_in * n_mats;
      const int boxes = min(kDecOutBoxes, (d - ow * out_rows + kDecOutRows - 1) / kDecOutRows);
      uint64_t* bar = &bars[w & 1];
      if (lane == 0) ptx::mbar_expect_tx(bar, (uint32_t)(boxes * kDecOutRows * kDecJB * 2));
      __syncwarp();
      if (lane < boxes)
        ptx::tma_load_2d(ring + (w & 1) * kDecHalfBytes + lane * (kDecOutRows * kDecJB * 2), &tmWo, bar, jb * kDecJB,
                         ph * d + ow * out_rows + lane * kDecOutRows);
    }
  };
  if (warp == 0) {
    ptx::fence_proxy_async();
    if (total > 0) issue_item_wave();
    if (total > 1) issue_item_wave();
  }

  if (blockIdx.x == gridDim.x - 1 && alive) {
    // ---------------------------------------------------------------- report (one CTA)
#pragma unroll 1
    for (int i = tid; i < T * E; i += kDecThreads) {
      const int t = i / E, e = i - t * E;
      a.logits[i] = slog[t * (kMaxE + 1) + e];
    }
    if (tid < P) {
      a.uidx[tid] = R->ue[tid]; a.ugate[tid] = R->ug[tid];
      a.midx[tid] = R->me[tid]; a.mgate[tid] = R->mg[tid];
      a.slot[tid] = R->sl[tid];
      a.perm[R->q[tid]] = tid;
      a.inv[tid] = R->q[tid];
    }
    if (tid < T) a.xnorm[tid] = R->xn[tid];
    if (tid <= K) {
      // per-slot counts and offsets over all K slots (the work items above only need the touched ones)
      int c = 0, lower = 0;
#pragma unroll 1
      for (int p = 0; p < P; ++p) { c += (R->sl[p] == tid); lower += (R->sl[p] < tid); }
      a.offset[tid] = lower;
      if (tid < K) a.count[tid] = c;
      if (tid < K && c > 0 && a.touched != nullptr) atomicAdd(a.touched, 1ull);   // slots whose weights were read
    }
    if (tid < K) {
      // Eq. (1) under the masked routing, credited to the slot's expert
      float m = 0.f;
#pragma unroll 1
      for (int p = 0; p < P; ++p)
        if (R->sl[p] == tid) m += R->xn[p / k] * fabsf(R->mg[p]) * a.enorm[R->me[p]];
      a.mimp[a.s2e[tid]] += m;
    }
    if (tid == kDecThreads - 1 && a.recent != nullptr) {
      // most-recent-first list of served experts: this step's (in slot order), then the older ones
      int old[kDecRecent], nw[kDecRecent];
#pragma unroll
      for (int h = 0; h < kDecRecent; ++h) { old[h] = a.recent[h]; nw[h] = -1; }
      int n = 0, hits = 0;
      for (int i = 0; i < R->n_touched; ++i) {
        const int e = R->me[R->pair_at[R->toffset[i]]];
        bool predicted = false;
#pragma unroll
        for (int h = 0; h < kDecRecent; ++h) predicted = predicted || (h < a.pf_depth && old[h] == e);
        hits += predicted ? 1 : 0;
        if (n < kDecRecent) nw[n++] = e;
      }
#pragma unroll
      for (int h = 0; h < kDecRecent; ++h) {
        bool dup = old[h] < 0;
#pragma unroll
        for (int q = 0; q < kDecRecent; ++q) dup = dup || (q < n && nw[q] == old[h]);
        if (!dup && n < kDecRecent) nw[n++] = old[h];
      }
#pragma unroll
      for (int h = 0; h < kDecRecent; ++h) a.recent[h] = nw[h];
      if (a.pf_stats != nullptr) {
        atomicAdd(a.pf_stats, (unsigned long long)hits);
        atomicAdd(a.pf_stats + 1, (unsigned long long)R->n_touched);
      }
    }
    if (tid < E) {
      // Eq. (1): terms of the off-the-shelf routing, added in pair order
      float s = 0.f;
      int n = 0;
      const float en = a.enorm[tid];
#pragma unroll 1
      for (int p = 0; p < P; ++p)
        if (R->ue[p] == tid) { s += R->xn[p / k] * fabsf(R->ug[p]) * en; ++n; }
      a.imp[tid] += s;
      a.cnt[tid] += (float)n;
    }
  }

  float yacc[kDecOutBoxes][4];      // a run's partial output rows: tile warp + 16 i, mma accumulator layout
  int run_jb = -1;                  // first hidden block of the current run, -1 = none open
  // consumer cursor: item index, wave inside the item, slot index, hidden block
  int it = 0, wi = 0, ti = n_items > 0 ? item0 / n_jb : 0, jb = n_items > 0 ? item0 - ti * n_jb : 0;
#pragma unroll 1
  for (int v = 0; v < total; ++v, ++wi) {
    if (wi == wpi) {                            // next item
      wi = 0;
      ++it;
      if (++jb == n_jb) { jb = 0; ++ti; }
    }
    const int s = R->touched[ti], n_s = R->tcount[ti], q0 = R->toffset[ti];
    const int grp = jb / kDecGroup;
    // runs need the whole output in one wave and all the slot's pairs in one mma
    const bool runs = n_out == 1 && n_s <= 8;
    // the run ends with this item unless the CTA's next item is in the same slot and group
    const bool run_ends = !runs || it + 1 >= my_items || jb + 1 == n_jb || (jb + 1) / kDecGroup != grp;
    const int w = n_rw + v;
    if (!dec_wait_wave(bars, w, R, a.status, 22)) { alive = false; break; }
    if (tid == 0 && v == 0) SWAPMOE_STAMP(0, 6);
    const unsigned char* st = ring + (w & 1) * kDecHalfBytes;
    if (wi < n_in * n_mats) {
      // ---- RW of the item's 32 hidden units: raw products W1 x (and W3 x), eight pairs at a time
      const int mat = wi >= n_in ? 1 : 0, rp = wi - mat * n_in;
#pragma unroll 1
      for (int nb = 0; nb < n_s; nb += 8) {
        const int nn = min(8, n_s - nb);
        if (tid < 8) R->tok[tid] = R->tok_at[q0 + nb + min(tid, nn - 1)];
        __syncthreads();
        dec_wave_dots(st, RW, d, xs, R, nn, red, (mat == 0 ? hraw : hraw3) + nb * kDecJB + rp * RW, kDecJB, RW);
      }
      if (wi == n_in * n_mats - 1) {
        // all 32 units of every pair are in: activation, rounded to bf16 for the second product
#pragma unroll 1
        for (int i = tid; i < n_s * kDecJB; i += kDecThreads) {
          const float v1 = hraw[i];
          const float h = a.swiglu ? v1 / (1.f + expf(-v1)) * hraw3[i] : fmaxf(v1, 0.f);
          hsb[(i / kDecJB) * kDecHPitch + (i % kDecJB)] = __float2bfloat16_rn(h);
        }
      }
    } else {
      // ---- up to 1024 rows of W_out's column slice (64 bytes per row, 64-byte swizzle): a warp
      // owns the 16-row tiles warp, warp + 16, ...; y[c][n] = sum_j W_out[c][j] h[n][j] over 32 j
      const int ow = wi - n_in * n_mats;
      const int g = lane >> 2, t = lane & 3;
#pragma unroll 1
      for (int nb = 0; nb < n_s; nb += 8) {
        const int nn = min(8, n_s - nb);
        const unsigned char* hrow = reinterpret_cast<const unsigned char*>(hsb) + (nb + min(g, nn - 1)) * (kDecHPitch * 2) + t * 4;
        const uint32_t b00 = lds32(hrow), b01 = lds32(hrow + 16), b10 = lds32(hrow + 32), b11 = lds32(hrow + 48);
        if (!runs || run_jb < 0) {              // a new run (without runs: every item, batch and wave)
          run_jb = jb;
#pragma unroll
          for (int i = 0; i < kDecOutBoxes; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) yacc[i][j] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < kDecOutBoxes; ++i) {
          const int r0 = (warp + kDecWarps * i) * 16 + g, r1 = r0 + 8;      // rows of the wave
          // 16-byte chunk j of row r sits at chunk j ^ ((r >> 1) & 3)
          const unsigned char* p0 = st + r0 * 64 + t * 4;
          const unsigned char* p1 = st + r1 * 64 + t * 4;
          const int x0 = (r0 >> 1) & 3, x1 = (r1 >> 1) & 3;
          mma_bf16_16x8x16(yacc[i], lds32(p0 + ((0 ^ x0) << 4)), lds32(p1 + ((0 ^ x1) << 4)), lds32(p0 + ((1 ^ x0) << 4)),
                           lds32(p1 + ((1 ^ x1) << 4)), b00, b01);
          mma_bf16_16x8x16(yacc[i], lds32(p0 + ((2 ^ x0) << 4)), lds32(p1 + ((2 ^ x1) << 4)), lds32(p0 + ((3 ^ x0) << 4)),
                           lds32(p1 + ((3 ^ x1) << 4)), b10, b11);
        }
        if (run_ends) {
          // partial rows of the run go out under the run's first hidden block
          float* yp = a.ypart + ((size_t)run_jb * P + q0 + nb) * d + ow * out_rows + g;
          const int n0 = 2 * t, n1 = 2 * t + 1;
#pragma unroll
          for (int i = 0; i < kDecOutBoxes; ++i) {
            const int c0 = (warp + kDecWarps * i) * 16;          // + g (in yp), + 8 for the second half
            if (ow * out_rows + c0 + g < d) {
              if (n0 < nn) yp[(size_t)n0 * d + c0] = yacc[i][0];
              if (n1 < nn) yp[(size_t)n1 * d + c0] = yacc[i][1];
            }
            if (ow * out_rows + c0 + g + 8 < d) {
              if (n0 < nn) yp[(size_t)n0 * d + c0 + 8] = yacc[i][2];
              if (n1 < nn) yp[(size_t)n1 * d + c0 + 8] = yacc[i][3];
            }
          }
        }
      }
    }
    const bool flush = wi == wpi - 1 && run_ends;
    __syncthreads();                              // the buffer is free; the activations are complete / free
    if (tid == 0 && v < 3) SWAPMOE_STAMP(0, 7 + v);
    if (warp == 0 && v + 2 < total) {
      ptx::fence_proxy_async();
      issue_item_wave();
    }
    if (!flush) continue;
    if (tid == 0) SWAPMOE_STAMP(0, 10);
    run_jb = -1;
    // ---- first-step sum: whoever delivers the group's last set of partial rows adds them all.
    // The group's sets: one per item, or with runs one per CTA whose item range meets the group
    // (CTA c holds items c*ipc ..; its set is filed under the first of them inside the group).
    const int g_first = grp * kDecGroup, g_size = min(kDecGroup, n_jb - g_first);
    const int gs = ti * n_jb + g_first;           // the group's first item, numbered over all items
    const int c_lo = gs / ipc, c_hi = (gs + g_size - 1) / ipc;
    const int n_sets = runs ? c_hi - c_lo + 1 : g_size;
    // One thread publishes for the whole CTA: the block barrier above ordered everybody's stores
    // before its fence (fences are cumulative), and its second fence orders the ticket before the
    // reads of the other CTAs' rows (L2 loads below).
    if (tid == 0) {
      __threadfence();
      const bool last = atomicAdd(&a.tickets[s * n_groups + grp], 1u) == (unsigned)(n_sets - 1);
      __threadfence();
      R->last = last;
    }
    __syncthreads();
    if (tid == 0) SWAPMOE_STAMP(0, 11);
    if (R->last) {
      const int d4 = d / 4;
      // thread (sub, col): sub = tid / 256 adds sets 8 sub .. 8 sub + 7 of 256 float4 columns (all eight
      // loads in flight together: one round trip per pair row at d_model 1024); the two sub-sums meet
      // in shared memory (the per-warp product area is free here) and are added in order
      const int sub = tid >> 8, col = tid & 255;
      float4* xch = reinterpret_cast<float4*>(red);       // [2][256] float4 = 8 KB
#pragma unroll 1
      for (int n = 0; n < n_s; ++n) {
#pragma unroll 1
        for (int c0 = 0; c0 < d4; c0 += 256) {
          const int c4 = c0 + col;
          float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
          if (c4 < d4) {
            float4 pv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int jj = sub * 8 + j;
              const int jbf = runs ? max(gs, (c_lo + jj) * ipc) - ti * n_jb : g_first + jj;   // where set jj was filed
              pv[j] = jj < n_sets ? __ldcg(reinterpret_cast<const float4*>(a.ypart + ((size_t)jbf * P + q0 + n) * d) + c4)
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) { sum.x += pv[j].x; sum.y += pv[j].y; sum.z += pv[j].z; sum.w += pv[j].w; }
          }
          xch[sub * 256 + col] = sum;
          __syncthreads();
          if (sub == 0 && c4 < d4) {
            const float4 o = xch[256 + col];
            sum.x += o.x; sum.y += o.y; sum.z += o.z; sum.w += o.w;
            reinterpret_cast<float4*>(a.gpart + ((size_t)grp * P + q0 + n) * d)[c4] = sum;
          }
          __syncthreads();
        }
      }
      __syncthreads();
      if (tid == 0) {
        SWAPMOE_STAMP(0, 12);
        a.tickets[s * n_groups + grp] = 0u;
        __threadfence();
        const bool last = atomicAdd(&a.tickets[K * n_groups], 1u) == (unsigned)(R->n_touched * n_groups - 1);
        __threadfence();
        R->last = last;
      }
      __syncthreads();
      if (R->last) {
        // ---- second step: all groups are in; gate-weighted sum into out (Section 2's combine)
#pragma unroll 1
        for (int t = 0; t < T; ++t) {
#pragma unroll 1
          for (int c4 = tid; c4 < d4; c4 += kDecThreads) {
          float o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
          for (int j = 0; j < k; ++j) {
            const int p = t * k + j, qq = R->q[p];
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int g2 = 0; g2 < n_groups; ++g2) {
              const float4 gv = __ldcg(reinterpret_cast<const float4*>(a.gpart + ((size_t)g2 * P + qq) * d) + c4);
              sum.x += gv.x; sum.y += gv.y; sum.z += gv.z; sum.w += gv.w;
            }
            const float gt = R->mg[p];
            o[0] = fmaf(gt, sum.x, o[0]); o[1] = fmaf(gt, sum.y, o[1]);
            o[2] = fmaf(gt, sum.z, o[2]); o[3] = fmaf(gt, sum.w, o[3]);
          }
          store4(a.out + (size_t)t * d + c4 * 4, o);
          }
        }
        if (tid == 0) a.tickets[K * n_groups] = 0u;
#ifdef SWAPMOE_TRACE
        __syncthreads();
        if (tid == 0) SWAPMOE_STAMP(0, 14);
#endif
      }
    }
    __syncthreads();     // R->last is reused by the next item
  }
  if (tid == 0) SWAPMOE_STAMP(0, 15);
  if (!alive && tid == 0) {
    // a wait gave up: let copies that may still be in flight land before the shared memory is released
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
}

inline cudaError_t decode_fused_set_smem_limit(int bytes) {
  return cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

}  // namespace swapmoe
