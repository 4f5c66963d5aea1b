// Slot histogram scan, stable token permutation, row gather and the importance
// reduction (SwapMoE Section 2: every token may pick a different expert; Eq. 1).
#pragma once
#include "common.cuh"

namespace swapmoe {

struct ScanArgs {
  const int32_t* cta_hist;   // [n_cta, K]
  const float* cta_imp;      // [n_cta, E]
  const float* cta_cnt;      // [n_cta, E] unmasked selections per expert (token counts), or nullptr
  const float* cta_mimp;     // [n_cta, K] Eq. (1) terms of the MASKED routing per slot, or nullptr
  const int32_t* s2e;        // [K] expert served by each slot (for cta_mimp)
  float* cnt;                // [E] accumulator of the token counts ("simple scheduling" score)
  float* mimp;               // [E] accumulator of Eq. (1) over the masked routing
  const int32_t* phys_slot;  // [K]
  int32_t* cta_base;         // [n_cta, K] pairs of the same slot in earlier CTAs (written only by the last-CTA scan)
  int32_t* count;            // [K]
  int32_t* offset;           // [K+1]  exclusive scan of count
  int32_t* pad_offset;       // [K+1]  same with every segment rounded up to kSegAlign rows
  TileDesc* tiles;           // GEMM work list
  int32_t* n_tiles;          // [1]
  float* imp;                // [E] accumulator of Eq. (1)
  unsigned* ticket;          // [1] router CTAs finished so far (returns to 0); nullptr: the router CTAs do not
                             // scan at all - the permute kernel sums the histograms itself (see below)
  TileDesc* tiles_b;         // optional second work list with tile_rows_b rows per tile (or nullptr)
  int32_t* n_tiles_b;
  unsigned long long* touched;   // [1] running total of slots that received at least one pair, or nullptr
  int32_t n_cta, K, E, tile_rows, tile_rows_b;
};

// Eq. (1) partial sums are added with ONE association wherever they are reduced: the router CTAs
// are cut into shares of kRedShare consecutive CTAs, a share is summed in CTA order, and the shares
// are added in order.  Whether one thread walks a column alone or the shares are summed side by
// side, the result is the same to the last bit, run to run and path to path.
constexpr int kRedShare = 16;

__device__ __forceinline__ float reduce_column_serial(const float* src, int n_rows, int C, int col) {
  float total = 0.f;
  for (int r0 = 0; r0 < n_rows; r0 += kRedShare) {
    const int r1 = min(n_rows, r0 + kRedShare);
    float acc = 0.f;
#pragma unroll 8
    for (int r = r0; r < r1; ++r) acc += src[(size_t)r * C + col];
    total += acc;
  }
  return total;
}

// Slot layout by one warp from the per-slot counts in shared memory: lane l owns slots l and l + 32
// (K <= 64); offsets, padded offsets and first-tile indices are exclusive prefix sums over the slots,
// taken with warp scans (tile heights are powers of two: shifts, no divisions - this code runs once,
// every dependent instruction counts).  s_off / s_pad (shared, may be nullptr) receive the exclusive
// offsets; with `write_global` the warp also writes count / offset / pad_offset and the tile lists.
__device__ __forceinline__ void slot_layout_warp(const ScanArgs& a, const int32_t* s_count, int32_t* s_off,
                                                 int32_t* s_pad, bool write_global) {
  const int lane = threadIdx.x & 31;
  const int sh_a = 31 - __clz(a.tile_rows);
  const bool two_lists = write_global && a.tiles_b != nullptr;
  const int sh_b = two_lists ? 31 - __clz(a.tile_rows_b) : 0;
  int c[2], off[2], pad[2], ta[2], tb[2], ph[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int s = lane + 32 * h;
    c[h] = s < a.K ? s_count[s] : 0;
    ph[h] = (write_global && s < a.K) ? a.phys_slot[s] : 0;     // issued early: its latency hides behind the scans
    off[h] = c[h];
    pad[h] = (c[h] + kSegAlign - 1) & ~(kSegAlign - 1);
    ta[h] = (c[h] + a.tile_rows - 1) >> sh_a;
    tb[h] = two_lists ? (c[h] + a.tile_rows_b - 1) >> sh_b : 0;
  }
  {
    // slots whose weights this forward reads: the algorithmic weight traffic of the layer
    const int nz = __popc(__ballot_sync(0xffffffffu, c[0] > 0)) + __popc(__ballot_sync(0xffffffffu, c[1] > 0));
    if (write_global && lane == 0 && a.touched != nullptr) atomicAdd(a.touched, (unsigned long long)nz);
  }
  // inclusive scans of the four quantities over 64 slots
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u0 = __shfl_up_sync(0xffffffffu, off[h], o), u1 = __shfl_up_sync(0xffffffffu, pad[h], o);
      const int u2 = __shfl_up_sync(0xffffffffu, ta[h], o), u3 = __shfl_up_sync(0xffffffffu, tb[h], o);
      if (lane >= o) { off[h] += u0; pad[h] += u1; ta[h] += u2; tb[h] += u3; }
    }
  }
  {
    const int t0 = __shfl_sync(0xffffffffu, off[0], 31), t1 = __shfl_sync(0xffffffffu, pad[0], 31);
    const int t2 = __shfl_sync(0xffffffffu, ta[0], 31), t3 = __shfl_sync(0xffffffffu, tb[0], 31);
    off[1] += t0; pad[1] += t1; ta[1] += t2; tb[1] += t3;
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int s = lane + 32 * h;
    if (s < a.K) {
      const int cnt = c[h];
      const int padded = (cnt + kSegAlign - 1) & ~(kSegAlign - 1);
      const int nt = (cnt + a.tile_rows - 1) >> sh_a;
      const int o_excl = off[h] - cnt, p_excl = pad[h] - padded, t_excl = ta[h] - nt;
      if (s_off != nullptr) { s_off[s] = o_excl; s_pad[s] = p_excl; }
      if (!write_global) continue;
      a.count[s] = cnt;
      a.offset[s] = o_excl;
      a.pad_offset[s] = p_excl;
      for (int i = 0; i < nt; ++i) {
        TileDesc td;
        td.phys = ph[h];
        td.row0 = p_excl + i * a.tile_rows;
        td.rows = min(a.tile_rows, cnt - i * a.tile_rows);
        td.slot = s;
        a.tiles[t_excl + i] = td;
      }
      if (s == a.K - 1) {
        a.offset[a.K] = off[h];
        a.pad_offset[a.K] = pad[h];
        *a.n_tiles = ta[h];
      }
      if (two_lists) {                         // same segments cut into tiles of another height
        const int ntb = (cnt + a.tile_rows_b - 1) >> sh_b;
        const int tb_excl = tb[h] - ntb;
        for (int i = 0; i < ntb; ++i) {
          TileDesc td;
          td.phys = ph[h];
          td.row0 = p_excl + i * a.tile_rows_b;
          td.rows = min(a.tile_rows_b, cnt - i * a.tile_rows_b);
          td.slot = s;
          a.tiles_b[tb_excl + i] = td;
        }
        if (s == a.K - 1) *a.n_tiles_b = tb[h];
      }
    }
  }
}

// Last-CTA form of the scan (routing without a permutation: swapmoe_route_static; grids of more
// than 256 router CTAs).  All threads of the LAST router CTA to finish call this: thread s walks
// slot s over the router CTAs in order (writing the running counts, `cta_base`, when asked), thread
// e adds expert e's Eq. (1) partials, then warp 0 lays out the slots.  The per-CTA arrays are first
// staged into shared memory with L1-bypassing copies when `stage` is large enough.
__device__ __forceinline__ void scan_reduce_block(const ScanArgs& a, void* stage, int stage_bytes) {
  __shared__ int32_t s_count[kMaxSlots];
  const int tid = threadIdx.x;
  // The accumulators' old values are fetched first so that their latency overlaps the staging
  // (thread e owns expert e, thread sl owns slot sl; blockDim.x >= E, K).
  const bool own_e = tid < a.E, own_s = tid < a.K;
  const float old_imp = own_e ? a.imp[tid] : 0.f;
  const float old_cnt = (own_e && a.cta_cnt) ? a.cnt[tid] : 0.f;
  const int my_expert = (own_s && a.cta_mimp) ? a.s2e[tid] : 0;
  const int n_hist = a.n_cta * a.K, n_imp = a.n_cta * a.E;
  const int n_cnt = a.cta_cnt ? n_imp : 0, n_mimp = a.cta_mimp ? n_hist : 0;
  const int32_t* hist = a.cta_hist;
  const float* impp = a.cta_imp;
  const float* cntp = a.cta_cnt;
  const float* mimpp = a.cta_mimp;
  if (stage != nullptr && (size_t)(n_hist + n_imp + n_cnt + n_mimp + 16) * 4 <= (size_t)stage_bytes &&
      (reinterpret_cast<uintptr_t>(stage) & 15) == 0) {
    // All four arrays are copied with 16-byte cp.async.cg (L2 only, no L1 allocation, no register
    // round trip), issued back to back: one memory latency in total.  Tails shorter than 16 bytes
    // are read with plain L1-bypassing loads.
    int32_t* sh = static_cast<int32_t*>(stage);
    float* si = reinterpret_cast<float*>(sh + ((n_hist + 3) & ~3));
    float* sc = si + ((n_imp + 3) & ~3);
    float* sm = sc + ((n_cnt + 3) & ~3);
    const void* srcs[4] = {a.cta_hist, a.cta_imp, a.cta_cnt, a.cta_mimp};
    void* dsts[4] = {sh, si, sc, sm};
    const int counts[4] = {n_hist, n_imp, n_cnt, n_mimp};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int n16 = counts[q] >> 2;
      const uint4* src = static_cast<const uint4*>(srcs[q]);
      const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(dsts[q]));
      for (int i = tid; i < n16; i += blockDim.x)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * i), "l"(src + i) : "memory");
      for (int i = (n16 << 2) + tid; i < counts[q]; i += blockDim.x)
        static_cast<int32_t*>(dsts[q])[i] = __ldcg(static_cast<const int32_t*>(srcs[q]) + i);
    }
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    hist = sh;
    impp = si;
    if (n_cnt) cntp = sc;
    if (n_mimp) mimpp = sm;
  }
  // Slots are walked by the LAST K threads and experts by the first E threads, so the two
  // chains run side by side.
  {
    const int s = (int)blockDim.x - 1 - tid;
    if (s < a.K) {
      int running = 0;
#pragma unroll 16
      for (int c = 0; c < a.n_cta; ++c) {
        const int v = hist[(size_t)c * a.K + s];
        if (a.cta_base != nullptr) a.cta_base[(size_t)c * a.K + s] = running;
        running += v;
      }
      s_count[s] = running;
    }
  }
  if (own_e) {
    a.imp[tid] = old_imp + reduce_column_serial(impp, a.n_cta, a.E, tid);
    if (a.cta_cnt != nullptr)                // token counts: small integers, exact in fp32
      a.cnt[tid] = old_cnt + reduce_column_serial(cntp, a.n_cta, a.E, tid);
  }
  if (own_s && a.cta_mimp != nullptr)        // slots map to distinct experts: no two threads share a target
    a.mimp[my_expert] += reduce_column_serial(mimpp, a.n_cta, a.K, tid);
  __syncthreads();
  if (tid < 32) slot_layout_warp(a, s_count, nullptr, nullptr, true);
}

// Called by every thread of a router CTA after its partials are written.  With a ticket counter the
// CTA that draws the last ticket runs the scan (no CTA waits for another); without one the router
// CTAs are done: the permute kernel sums the per-CTA histograms itself.
__device__ __forceinline__ void finish_router_cta(const ScanArgs& a, void* stage = nullptr, int stage_bytes = 0) {
  if (threadIdx.x == 0) SWAPMOE_STAMP(0, 7);
  if (a.ticket == nullptr) return;
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned ticket = atomicAdd(a.ticket, 1u);
    s_last = (ticket == (unsigned)a.n_cta - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    scan_reduce_block(a, stage, stage_bytes);
    if (threadIdx.x == 0) *a.ticket = 0u;
    if (threadIdx.x == 0) SWAPMOE_STAMP(0, 9);
  }
}

struct PermuteArgs {
  const void* x;              // [T, d]
  const int32_t* slot;        // [T*k]
  const int32_t* cta_base;    // [n_cta, K] pairs of the same slot in earlier router CTAs  } read when the router's
  const int32_t* offset;      // [K+1]                                                      } last CTA scanned
  const int32_t* pad_offset;  // [K+1]                                                      } (own_scan == 0)
  int32_t* perm;              // [T*k]
  int32_t* inv;               // [T*k]
  int32_t* inv_pad;           // [T*k] row of the pair in the padded workspace
  int32_t* row_pair;          // [rows_pad] flat pair index stored in each occupied padded row
  void* xp;                   // [rows_pad, d]
  int32_t T, d, k, K, tok_tile;
  int32_t own_scan;           // 1: this kernel sums the router's per-CTA histograms itself (scan.*), CTA (0, 0)
                              // publishes count / offset / pad_offset / tile lists, and the extra CTA column
                              // blockIdx.x == scan.n_cta reduces the Eq. (1) partials
  ScanArgs scan;
};

constexpr int kPermThreads = 512;

// The Eq. (1) reduction of the forward (one CTA of the permute kernel, off everybody's critical path):
// work item (share, column) sums its kRedShare router CTAs in order; thread `column` then adds the
// shares in order - the association of reduce_column_serial.
__device__ __forceinline__ float reduce_columns_parallel(const float* src, int n_rows, int C, float* s_red,
                                                         int cap_floats) {
  const int tid = threadIdx.x;
  const int n_share = (n_rows + kRedShare - 1) / kRedShare;
  const int cols_per_pass = max(1, min(C, cap_floats / n_share));    // columns whose shares fit the buffer at once
  float total = 0.f;
  for (int c0 = 0; c0 < C; c0 += cols_per_pass) {
    const int nc = min(cols_per_pass, C - c0);
    for (int w = tid; w < n_share * nc; w += kPermThreads) {
      const int sh = w / nc, col = c0 + (w - sh * nc);
      const int r0 = sh * kRedShare, r1 = min(n_rows, r0 + kRedShare);
      float v[kRedShare];
#pragma unroll
      for (int u = 0; u < kRedShare; ++u) v[u] = r0 + u < r1 ? src[(size_t)(r0 + u) * C + col] : 0.f;   // all in flight together
      float acc = 0.f;
#pragma unroll
      for (int u = 0; u < kRedShare; ++u) acc += v[u];       // adding 0.f beyond the last row changes nothing
      s_red[w] = acc;
    }
    __syncthreads();
    if (tid >= c0 && tid < c0 + nc)
      for (int sh = 0; sh < n_share; ++sh) total += s_red[sh * nc + (tid - c0)];
    __syncthreads();
  }
  return total;
}

// One CTA = the pairs of tok_tile (<= 128) tokens in flat order p = t*k + j.  The rank of a
// pair among the pairs of the same slot is: pairs in earlier CTAs +
// pairs in earlier warps of this CTA + earlier lanes of this warp (match + popc),
// which is exactly a stable counting sort.  gridDim.y CTAs share one token tile: each
// recomputes the (cheap) positions and copies every gridDim.y-th row of the tile.
// The kernel is a chain of memory round trips, so the independent ones are started together:
// the token rows (inputs of the layer, so even before the wait on the predecessor) go to
// registers while the slots and the histograms are fetched.
//
// own_scan: the router CTAs only left their per-CTA slot histograms [n_cta, K].  Every CTA here adds
// the rows of all router CTAs (slot totals -> offsets) and of the router CTAs in front of its token
// tile (its base counts): thread (share, slot) adds a contiguous share of the rows, thread `slot` adds
// the shares.  That is 8 KB of L2 reads per CTA at 2048 tokens, in place of a serial scan by the last
// router CTA that kept every other SM waiting for a third of the router's duration.
template <typename T>
__global__ void __launch_bounds__(kPermThreads) permute_gather_kernel(const PermuteArgs a) {
  // 11 KB of shared memory, so that these CTAs fit beside a router CTA (over 210 KB) and are already
  // waiting when the router finishes.  The reducing CTAs use the same bytes for their shares.
  constexpr int kRawBytes = (kPermThreads / 32) * kMaxSlots * 4 + kPermThreads * 4 + 4 * kMaxSlots * 4 + 2 * kPermThreads * 4;
  __shared__ __align__(16) unsigned char s_raw[kRawBytes];
  int32_t (*wcount)[kMaxSlots] = reinterpret_cast<int32_t (*)[kMaxSlots]>(s_raw);
  int32_t* dst_row = reinterpret_cast<int32_t*>(s_raw + (kPermThreads / 32) * kMaxSlots * 4);
  int32_t* s_base = dst_row + kPermThreads;
  int32_t* s_off = s_base + kMaxSlots;
  int32_t* s_pad = s_off + kMaxSlots;
  int32_t* s_tot = s_pad + kMaxSlots;
  int32_t (*s_part)[kPermThreads] = reinterpret_cast<int32_t (*)[kPermThreads]>(s_tot + kMaxSlots);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // the next kernel's CTAs may be scheduled at once: they stop at their own wait, and until then they
  // touch nothing this kernel or the router writes
  pdl_trigger();
  if (a.own_scan && (int)blockIdx.x >= a.scan.n_cta) {
    // ---- the three extra columns of CTAs: the first CTA of column n_cta + w reduces score w of {Eq. (1), token
    // counts, Eq. (1) over the masked routing}: each is done before the copying CTAs are, none delays the grid
    if (blockIdx.y != 0) return;
    const ScanArgs& sc = a.scan;
    pdl_wait();
    float* s_red = reinterpret_cast<float*>(s_raw);
    {
      const int which = (int)blockIdx.x - sc.n_cta;
      if (tid == 0) SWAPMOE_STAMP(1, 4 + 2 * which);
      const float* src = which == 0 ? sc.cta_imp : which == 1 ? sc.cta_cnt : sc.cta_mimp;
      if (src == nullptr) return;
      const int C = which == 2 ? sc.K : sc.E;
      float* acc = which == 0 ? sc.imp : which == 1 ? sc.cnt : sc.mimp;
      // thread c owns column c: expert c, or for the masked score the expert that slot c serves
      const int target = tid < C ? (which == 2 ? sc.s2e[tid] : tid) : 0;
      const float old = tid < C ? acc[target] : 0.f;
      const float v = reduce_columns_parallel(src, sc.n_cta, C, s_red, kRawBytes / 4);
      if (tid < C) acc[target] = old + v;
      if (tid == 0) SWAPMOE_STAMP(1, 5 + 2 * which);
    }
    return;
  }
  if (tid == 0 && blockIdx.y == 0) SWAPMOE_STAMP(1, 0);
  const int npair = a.tok_tile * a.k;          // <= 512
  const int nwarp_p = (npair + 31) >> 5;
  const int p0 = blockIdx.x * npair;
  const int n_total = a.T * a.k;

  for (int i = lane; i < kMaxSlots; i += 32) wcount[warp][i] = 0;     // each warp clears (and later fills) its own row
  __syncwarp();
  // this CTA's rows: local pair pl = ri * gridDim.y + blockIdx.y; the first kPre 16-byte pieces per
  // thread are fetched now
  constexpr int kPre = 4;
  const int vec_per_row = a.d * (int)sizeof(T) / 16;
  const uint4* src = static_cast<const uint4*>(a.x);
  const int my_rows = (npair - (int)blockIdx.y + (int)gridDim.y - 1) / (int)gridDim.y;
  uint4 pre[kPre];
#pragma unroll
  for (int u = 0; u < kPre; ++u) {
    const int i = tid + u * kPermThreads;
    pre[u] = make_uint4(0u, 0u, 0u, 0u);
    if (i < my_rows * vec_per_row) {
      const int ri = i / vec_per_row, v = i - ri * vec_per_row;
      const int pg = p0 + ri * (int)gridDim.y + (int)blockIdx.y;
      if (pg < n_total) pre[u] = src[(size_t)(pg / a.k) * vec_per_row + v];
    }
  }
  pdl_wait();
  if (tid == 0 && blockIdx.y == 0) SWAPMOE_STAMP(1, 1);
  int s = -1, rank = 0;
  const int p = p0 + tid;
  if (tid < npair && p < n_total) s = a.slot[p];
  if (a.own_scan) {
    // thread (share, slot): the histogram rows of a contiguous share of the router CTAs, all loads in flight together
    const int K = a.K, n_cta = a.scan.n_cta, n_before = (int)blockIdx.x;
    const int PK = kPermThreads / K;                       // shares per slot
    const int R = (n_cta + PK - 1) / PK;                   // router CTAs per share (<= 8 up to 256 CTAs, K = 16)
    const int sh = tid / K, col = tid - sh * K;
    if (sh < PK) {
      int tot = 0, before = 0;
      const int c0 = sh * R, c1 = min(n_cta, c0 + R);
      for (int cb = c0; cb < c1; cb += 8) {
        int v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = cb + u < c1 ? a.scan.cta_hist[(size_t)(cb + u) * K + col] : 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) { tot += v[u]; before += cb + u < n_before ? v[u] : 0; }
      }
      s_part[0][tid] = tot;
      s_part[1][tid] = before;
    }
    if (warp < nwarp_p) {                      // ranks inside the warp need only the pairs' slots
      const uint32_t same = __match_any_sync(0xffffffffu, s);
      rank = __popc(same & ((1u << lane) - 1u));
      if (s >= 0 && rank == 0) wcount[warp][s] = __popc(same);
    }
    __syncthreads();
    if (tid < K) {
      int tot = 0, before = 0;
#pragma unroll 8
      for (int q = 0; q < PK; ++q) { tot += s_part[0][q * K + tid]; before += s_part[1][q * K + tid]; }
      s_tot[tid] = tot;
      s_base[tid] = before;
    }
    __syncthreads();
    if (warp == 0) slot_layout_warp(a.scan, s_tot, s_off, s_pad, blockIdx.x == 0 && blockIdx.y == 0);
  } else {
    if (tid < a.K) {
      s_base[tid] = a.cta_base[(size_t)blockIdx.x * a.K + tid];
      s_off[tid] = a.offset[tid];
      s_pad[tid] = a.pad_offset[tid];
    }
    if (warp < nwarp_p) {
      const uint32_t same = __match_any_sync(0xffffffffu, s);
      rank = __popc(same & ((1u << lane) - 1u));
      if (s >= 0 && rank == 0) wcount[warp][s] = __popc(same);
    }
  }
  __syncthreads();
  if (s >= 0) {
    int before = s_base[s];
    for (int w = 0; w < warp; ++w) before += wcount[w][s];
    const int within = before + rank;
    const int pos = s_off[s] + within;
    const int row = s_pad[s] + within;
    if (blockIdx.y == 0) {
      a.perm[pos] = p;
      a.inv[p] = pos;
      a.inv_pad[p] = row;
      a.row_pair[row] = p;
    }
    dst_row[tid] = row;
  } else if (tid < npair) {
    dst_row[tid] = -1;
  }
  __syncthreads();
  if (tid == 0 && blockIdx.y == 0) SWAPMOE_STAMP(1, 2);
  // Gather: copy each pair's token row into its slot segment, 16 bytes per access.
  uint4* dst = static_cast<uint4*>(a.xp);
#pragma unroll
  for (int u = 0; u < kPre; ++u) {
    const int i = tid + u * kPermThreads;
    if (i < my_rows * vec_per_row) {
      const int ri = i / vec_per_row, v = i - ri * vec_per_row;
      const int row = dst_row[ri * gridDim.y + blockIdx.y];
      if (row >= 0) dst[(size_t)row * vec_per_row + v] = pre[u];
    }
  }
  for (int i = tid + kPre * kPermThreads; i < my_rows * vec_per_row; i += kPermThreads) {
    const int ri = i / vec_per_row, v = i - ri * vec_per_row;
    const int pl = ri * gridDim.y + blockIdx.y;
    const int row = dst_row[pl];
    if (row >= 0) {
      const int t = (p0 + pl) / a.k;
      dst[(size_t)row * vec_per_row + v] = src[(size_t)t * vec_per_row + v];
    }
  }
  if (tid == 0 && blockIdx.y == 0) SWAPMOE_STAMP(1, 3);
}

struct CombineArgs {
  const float* y;            // [rows_pad, d] fp32 expert outputs
  const int32_t* inv_pad;    // [T*k]
  const float* mgate;        // [T*k]
  void* out;                 // [T, d]
  long long split_stride;    // elements between the copies of y
  int32_t T, d, k, n_split;  // n_split copies of y hold partial sums that are added here, in order
};

// out[t, c] = sum_j mgate[t,j] * y[inv_pad[t,j], c]; each thread owns 8 columns.
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(const CombineArgs a) {
  pdl_wait();
  pdl_trigger();
  const int c8n = a.d >> 3;
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= (long long)a.T * c8n) return;
  const int t = (int)(idx / c8n), c = (int)(idx - (long long)t * c8n) * 8;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int j = 0; j < a.k; ++j) {
    const float g = a.mgate[(size_t)t * a.k + j];
    const float* yr = a.y + (size_t)a.inv_pad[(size_t)t * a.k + j] * a.d + c;
    float4 y0 = reinterpret_cast<const float4*>(yr)[0];
    float4 y1 = reinterpret_cast<const float4*>(yr)[1];
    for (int z = 1; z < a.n_split; ++z) {
      const float4 p0 = reinterpret_cast<const float4*>(yr + (size_t)z * a.split_stride)[0];
      const float4 p1 = reinterpret_cast<const float4*>(yr + (size_t)z * a.split_stride)[1];
      y0.x += p0.x; y0.y += p0.y; y0.z += p0.z; y0.w += p0.w;
      y1.x += p1.x; y1.y += p1.y; y1.z += p1.z; y1.w += p1.w;
    }
    acc[0] = fmaf(g, y0.x, acc[0]); acc[1] = fmaf(g, y0.y, acc[1]);
    acc[2] = fmaf(g, y0.z, acc[2]); acc[3] = fmaf(g, y0.w, acc[3]);
    acc[4] = fmaf(g, y1.x, acc[4]); acc[5] = fmaf(g, y1.y, acc[5]);
    acc[6] = fmaf(g, y1.z, acc[6]); acc[7] = fmaf(g, y1.w, acc[7]);
  }
  store8(static_cast<T*>(a.out) + (size_t)t * a.d + c, acc);
}

// Installs the slot tables (arguments travel by value in the launch, so the host
// arrays may be reused immediately and earlier forwards keep the old tables).
struct SlotTables {
  int32_t e2s[kMaxE];
  int32_t phys[kMaxSlots];
  int32_t s2e[kMaxSlots];
};
static __global__ void set_tables_kernel(const SlotTables t, int E, int K, int32_t* e2s, int32_t* phys,
                                  int32_t* s2e) {
  for (int i = threadIdx.x; i < E; i += blockDim.x) e2s[i] = t.e2s[i];
  for (int i = threadIdx.x; i < K; i += blockDim.x) { phys[i] = t.phys[i]; s2e[i] = t.s2e[i]; }
}

}  // namespace swapmoe
