// C ABI of the Virtual-Expert MoE-layer forward (see include/swapmoe.h): argument
// checks, workspace layout and kernel launches.  No host synchronisation and no
// allocation happen inside forward().
#include "../../include/swapmoe.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"
#include "decode_fused.cuh"
#include "gemm_mma.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc_f32.cuh"
#include "gemm_tc_pair.cuh"
#include "gemm_tc_ffn.cuh"
#include "gemm_tc_small.cuh"
#include "permute.cuh"
#include "router_gate.cuh"
#include "router_tc.cuh"
#include "router_small.cuh"
#include "router_small_f32.cuh"

using namespace swapmoe;

struct swapmoe_layer {
  swapmoe_config_t cfg;
  int device;
  int nin;
  size_t elem;
  // device workspace (one allocation)
  char* ws_base;
  size_t ws_bytes;
  float *logits, *ugate, *mgate, *xnorm, *cta_imp, *cta_cnt, *cta_mimp, *imp, *cnt, *mimp, *enorm, *y;
  int32_t *uidx, *midx, *slot, *cta_hist, *cta_base, *count, *offset, *pad_offset;
  int32_t *perm, *inv, *inv_pad, *row_pair, *n_tiles, *e2s, *phys, *s2e, *status;
  unsigned* ticket;
  int32_t* dec_recent;         // one-launch decode path: experts served most recently (device)
  unsigned long long* dec_pf_stats;   // ... and how often its L2 prefetch of them was right (device)
  int32_t dec_pf_depth;        // recently served experts to prefetch while routing (SWAPMOE_DECODE_PREFETCH, 0 = off)
  unsigned long long* touched; // running total of slots that received at least one pair (device)
  bool small_path;             // small-batch GEMM kernels for <= 64 pairs
  TcSmallCache small;
  TileDesc* tiles;
  TileDesc* tiles_b;           // 128-row work list kept beside a 256-row one (see forward_impl)
  int32_t* n_tiles_b;
  void *xp, *h, *x_stage, *out_stage;
  // host state
  const void *Wr, *arena_in, *arena_out;
  bool router_set, resident_set;
  int32_t h_s2e[kMaxSlots], h_phys[kMaxSlots];
  int32_t last_T;
  int64_t launches;
  int32_t gemm_path;
  int32_t rows_pad_max;
  int pair_min_rows;           // ... used when the slots hold at least this many rows on average (SWAPMOE_PAIR_MIN_ROWS)
  int gemm_pairs;              // CTA pairs available to the cta_group::2 grouped GEMM (0: not used; SWAPMOE_PAIR_GEMM=0)
  bool small_router_f32;       // fp32 layers: eight-token CTAs of the split-TF32 mma router (SWAPMOE_SMALL_ROUTER=0: never)
  bool small_router;           // eight-token mma router CTAs for batches of up to 64 tokens (bf16)
  int32_t small_router_max_t;  // ... and sixteen-token CTAs up to this many tokens (0: never)
  bool decode_path;            // one-launch forward for a handful of tokens (bf16)
  int32_t decode_max_pairs;    // ... used up to this many (token, expert) pairs (the kernel takes 8 tokens)
  float* dec_ws;               // its partial-row workspace
  unsigned* dec_tickets;
  CUtensorMap dec_map_wo;      // W_out viewed for the decode kernel's column-slice loads
  int row_group;               // row tiles per scheduling group of the grouped GEMMs (0: automatic; SWAPMOE_ROW_GROUP)
  bool h_valid, y_valid;       // whether the last forward left h / y in the workspace (debug taps)
  int32_t y_split_last;        // copies of y the last forward's GEMM-2 wrote (slices of its contraction)
  int32_t rerun_gemm;          // 0, or the grouped GEMM swapmoe_debug_rerun_gemm is re-launching (1 / 2)
  int32_t permute_groups;      // 0 = automatic, else row groups (CTAs per token tile) of the permute kernel
  int32_t y_copies;            // copies of y in the workspace (slices of a split contraction)
  int32_t sm_count;
  bool use_pdl;                // programmatic dependent launch between the kernels of a forward
  cudaStream_t s_in, s_out;    // private copy streams of the asynchronous host path
  cudaEvent_t ev_in, ev_comp, ev_out, ev_load;
  int32_t router_tok;          // 0 = automatic token-tile size of the tensor-core router, else 32/64/128
  bool prefetch;               // pull resident weights into L2 from the router kernel
  long long l2_prefetch_bytes; // how much of them (L2 capacity minus head room)
  bool fp32_swap;              // fp32 layers: swapped-operand GEMM for small slots
  int prefetch_min_pairs;      // ... when the batch has at least this many HALF pairs per slot (SWAPMOE_PREFETCH_MIN_PAIRS)
  void* const* stage_events;   // 7 cudaEvent_t of the forward being enqueued, or nullptr
  CUtensorMap map_x;           // TMA view of the last token matrix [T, d]
  const void* map_x_ptr;
  int32_t map_x_T;
  TcState tc;
  TcF32State tc32;             // tcgen05 grouped GEMM of fp32 layers, bf16-piece split (SWAPMOE_FP32_TC=0: warp-level mma)
  PFN_encodeTiled encode32;
};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Carver {
  size_t off = 0;
  template <typename T>
  size_t take(size_t n) {
    const size_t o = off;
    off = align_up(off + n * sizeof(T), 256);
    return o;
  }
};

inline bool cuda_ok(cudaError_t e) { return e == cudaSuccess; }

// One small launch copies the selected per-expert scores of a layer into mapped pinned host memory and zeroes
// them: a pair of tiny memcpy / memset nodes per score costs 10-15 us of stream time each, which a decode step of
// a few hundred microseconds cannot afford twelve layers at a time.
struct ScoreSnapshot { float* acc[3]; float* dst; int E, mask, reset; };
__global__ void snapshot_scores_kernel(const ScoreSnapshot s) {
  for (int k = 0; k < 3; ++k) {
    if (!((s.mask >> k) & 1)) continue;
    for (int e = threadIdx.x; e < s.E; e += blockDim.x) {
      s.dst[k * s.E + e] = s.acc[k][e];
      if (s.reset) s.acc[k][e] = 0.f;
    }
  }
  __threadfence_system();
}

struct EnormTable { float v[kMaxE]; };
__global__ void set_enorm_kernel(const EnormTable t, int E, float* enorm) {
  for (int i = threadIdx.x; i < E; i += blockDim.x) enorm[i] = t.v[i];
}

inline void mark(swapmoe_layer* L, int i, cudaStream_t st) {
  if (L->stage_events) cudaEventRecord(static_cast<cudaEvent_t>(L->stage_events[i]), st);
}

int32_t check_launch() { return cuda_ok(cudaGetLastError()) ? SWAPMOE_OK : SWAPMOE_ERR_CUDA; }

template <typename DT>
int32_t forward_impl(swapmoe_layer* L, const void* x, const float* ext_logits, void* out, int32_t T,
                     cudaStream_t st) {
  const swapmoe_config_t& c = L->cfg;
  const bool pdl = L->use_pdl && L->stage_events == nullptr;
  const int rerun = L->rerun_gemm;          // 1 / 2: only that grouped GEMM, on the state the last forward left
  if (L->decode_path && T <= kDecMaxTokens && T * c.top_k <= L->decode_max_pairs && c.dtype == SWAPMOE_BF16) {
    if (rerun) return SWAPMOE_ERR_UNSUPPORTED;   // the one-launch kernel has no GEMM launch of its own
    // a handful of tokens: routing, both expert products and the combine in one launch
    DecodeArgs da;
    da.x = static_cast<const bf16*>(x); da.Wr = static_cast<const bf16*>(L->Wr); da.ext_logits = ext_logits;
    da.e2s = L->e2s; da.s2e = L->s2e; da.phys = L->phys; da.enorm = L->enorm;
    da.arena_in = static_cast<const bf16*>(L->arena_in); da.arena_out = static_cast<const bf16*>(L->arena_out);
    da.in_stride = (long long)L->nin * c.d_ff * c.d_model; da.out_stride = (long long)c.d_ff * c.d_model;
    da.logits = L->logits; da.uidx = L->uidx; da.ugate = L->ugate; da.midx = L->midx; da.mgate = L->mgate;
    da.slot = L->slot; da.xnorm = L->xnorm; da.count = L->count; da.offset = L->offset; da.perm = L->perm;
    da.inv = L->inv; da.imp = L->imp; da.cnt = L->cnt; da.mimp = L->mimp;
    const size_t n_jb = c.d_ff / kDecJB;
    da.ypart = L->dec_ws; da.gpart = L->dec_ws + n_jb * (size_t)(kDecMaxTokens * c.top_k) * c.d_model;
    da.tickets = L->dec_tickets; da.out = static_cast<bf16*>(out); da.status = L->status; da.touched = L->touched;
    da.recent = L->dec_recent; da.pf_stats = L->dec_pf_stats; da.pf_depth = L->dec_pf_depth;
    da.T = T; da.d = c.d_model; da.f = c.d_ff; da.E = c.E; da.k = c.top_k; da.K = c.K; da.renorm = c.renorm_topk;
    da.swiglu = c.act == SWAPMOE_ACT_SWIGLU;
    mark(L, 0, st);
    if (launch_kernel(decode_fused_kernel, dim3(L->sm_count), dim3(kDecThreads), decode_smem_bytes(c.d_model), st, pdl,
                      L->dec_map_wo, da) != cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    L->launches++;
    L->h_valid = L->y_valid = false;          // the one-launch kernel keeps both in shared memory
    for (int i = 1; i <= 6; ++i) mark(L, i, st);
    return check_launch();
  }
  const bool tc_router = L->tc.router_ok && ext_logits == nullptr;
  // up to 64 tokens: eight-token CTAs of the mma router (the tcgen05 router's fixed cost dominates there)
  // (and sixteen-token CTAs while they still fit one wave of CTAs)
  const int rs_nt = !(tc_router && L->small_router) ? 0 : (T <= kRsMaxTokens ? 1 : (T <= L->small_router_max_t ? 2 : 0));
  const bool small_router = rs_nt > 0;
  int tok_tile = tc_router ? router_tc_tok(T) : kTokTile;
  if (tc_router && L->router_tok) tok_tile = L->router_tok;
  if (small_router) tok_tile = kRsTok * rs_nt;
  // fp32 layers: eight-token CTAs of the split-TF32 mma router while they fit one wave of CTAs
  const bool small_f32 = L->small_router_f32 && ext_logits == nullptr && T <= kRsTok * std::min(L->sm_count, 256);
  if (small_f32) tok_tile = kRsTok;
  const int n_cta = (T + tok_tile - 1) / tok_tile;
  const int n_pairs = T * c.top_k;
  const bool use_tc = tc_selected(L->gemm_path, c, T);
  const bool use_pairs = use_tc && tc_use_pairs(c, T, L->gemm_pairs, L->pair_min_rows);
  const int mt = use_tc ? tc_row_subtiles(c, T, use_pairs) : 1;
  const bool use_tc32 = !use_tc && L->tc32.enabled && L->tc32.arena_bound;
  // fp32 layers whose slots hold well under 128 rows on average: weights on the MMA's rows, the slot's tokens on its
  // columns (64-token tiles), so that no tensor time goes to empty rows (SWAPMOE_FP32_SWAP=0: never)
  const bool swap32 = use_tc32 && L->tc32.swap_ok && L->fp32_swap && (long long)n_pairs < 96ll * c.K;
  const int tile_rows = use_tc ? kTcBM * mt : (use_tc32 ? (swap32 ? kF32SwapTok : kTcBM) : kMmaBM);
  const int max_tiles = (n_pairs + tile_rows - 1) / tile_rows + c.K;

  RouterArgs ra;
  ra.x = x; ra.Wr = L->Wr; ra.ext_logits = ext_logits; ra.e2s = L->e2s; ra.enorm = L->enorm;
  ra.logits = L->logits; ra.uidx = L->uidx; ra.ugate = L->ugate; ra.midx = L->midx;
  ra.mgate = L->mgate; ra.slot = L->slot; ra.xnorm = L->xnorm; ra.cta_hist = L->cta_hist;
  ra.cta_imp = L->cta_imp;
  ra.cta_cnt = L->cta_cnt; ra.cta_mimp = L->cta_mimp;
  ra.T = T; ra.d = c.d_model; ra.E = c.E; ra.k = c.top_k; ra.K = c.K; ra.renorm = c.renorm_topk;
  ScanArgs& sa = ra.scan;
  sa.cta_hist = L->cta_hist; sa.cta_imp = L->cta_imp; sa.phys_slot = L->phys;
  // Up to 256 router CTAs the router only leaves its per-CTA histograms and the permute kernel sums them itself
  // (every CTA its own base counts, one CTA the Eq. (1) partials); beyond that the last router CTA to finish scans
  // (re-reading all rows in every permute CTA would then cost more than its serial walk).
  const bool own_scan = n_cta <= 256;
  sa.cta_base = own_scan ? nullptr : L->cta_base; sa.count = L->count; sa.offset = L->offset;
  sa.pad_offset = L->pad_offset; sa.tiles = L->tiles; sa.n_tiles = L->n_tiles; sa.imp = L->imp;
  sa.cta_cnt = L->cta_cnt; sa.cta_mimp = L->cta_mimp; sa.s2e = L->s2e; sa.cnt = L->cnt; sa.mimp = L->mimp;
  sa.ticket = own_scan ? nullptr : L->ticket;
  sa.touched = L->touched;
  sa.n_cta = n_cta; sa.K = c.K; sa.E = c.E; sa.tile_rows = tile_rows;
  // GEMM-2 with two row sub-tiles per CTA walks 256-row tiles; GEMM-1 then gets its own compact
  // list of 128-row tiles (walking the 256-row list as pairs would leave holes in its schedule).
  sa.tiles_b = mt == 2 ? L->tiles_b : nullptr; sa.n_tiles_b = L->n_tiles_b; sa.tile_rows_b = kTcBM;
  ra.pf_base[0] = ra.pf_base[1] = nullptr;
  ra.pf_slot_bytes[0] = ra.pf_slot_bytes[1] = 16384;
  ra.pf_total_bytes[0] = ra.pf_total_bytes[1] = 0;
  ra.pf_phys = L->phys;
  int pf_ctas = 0;
  if (tc_router && use_tc && L->prefetch && 2 * n_pairs >= L->prefetch_min_pairs * c.K &&
      (long long)c.K * (L->nin + 1) * c.d_ff * c.d_model * (long long)L->elem <= (320ll << 20)) {
    // Most slots will be touched (at least half a pair per slot): pull the resident weights towards L2 now,
    // while the router and the permutation leave HBM idle (a slot that stays untouched costs idle bandwidth only).  GEMM-1's matrices first, then as much of GEMM-2's
    // as the L2 budget allows.
    const long long in_slot = (long long)L->nin * c.d_ff * c.d_model * L->elem;
    const long long out_slot = (long long)c.d_ff * c.d_model * L->elem;
    const long long budget = L->l2_prefetch_bytes;
    long long in_total = in_slot * c.K, out_total = out_slot * c.K;
    if (in_total > budget) in_total = budget / 16384 * 16384;
    if (out_total > budget - in_total) out_total = (budget - in_total) / 16384 * 16384;
    ra.pf_base[0] = static_cast<const char*>(L->arena_in);
    ra.pf_base[1] = static_cast<const char*>(L->arena_out);
    ra.pf_slot_bytes[0] = in_slot; ra.pf_slot_bytes[1] = out_slot;
    ra.pf_total_bytes[0] = in_total; ra.pf_total_bytes[1] = out_total;
    pf_ctas = L->sm_count - n_cta;
    if (pf_ctas < 0) pf_ctas = 0;
    if (pf_ctas > 64) pf_ctas = 64;
  }
  mark(L, 0, st);
  if (rerun) {
    // measurement re-run: routing, permutation and tile list are those of the last forward
  } else if (small_router) {
    if ((rs_nt == 1 ? launch_kernel(router_small_kernel<1>, dim3(n_cta + pf_ctas), dim3(kDecThreads),
                                    router_small_smem_bytes(c.d_model, 1), st, pdl, ra, L->status)
                    : launch_kernel(router_small_kernel<2>, dim3(n_cta + pf_ctas), dim3(kDecThreads),
                                    router_small_smem_bytes(c.d_model, 2), st, pdl, ra, L->status)) != cudaSuccess)
      return SWAPMOE_ERR_CUDA;
  } else if (tc_router) {
    if (x != L->map_x_ptr || T != L->map_x_T) {   // the token map is re-encoded only when x or T changes
      if (!tc_encode_2d(L->tc.encode, &L->map_x, x, (uint64_t)T, (uint64_t)c.d_model, (uint32_t)tok_tile))
        return SWAPMOE_ERR_CUDA;
      L->map_x_ptr = x;
      L->map_x_T = T;
    }
    if (launch_kernel(router_tc_kernel, dim3(n_cta + pf_ctas), dim3(kRtThreads), router_tc_smem_bytes(c.E, tok_tile),
                      st, pdl, L->map_x, L->tc.map_wr, ra, L->status, router_tc_stages(c.E, tok_tile), tok_tile) !=
        cudaSuccess)
      return SWAPMOE_ERR_CUDA;
  } else if (small_f32) {
    if (launch_kernel(router_small_f32_kernel, dim3(n_cta), dim3(kDecThreads), router_small_f32_smem_bytes(c.d_model), st,
                      pdl, ra, L->status) != cudaSuccess)
      return SWAPMOE_ERR_CUDA;
  } else {
    if (launch_kernel(router_gate_fn<DT>(c.E), dim3(n_cta), dim3(256), router_smem_bytes(c.E), st, pdl, ra) !=
        cudaSuccess)
      return SWAPMOE_ERR_CUDA;
  }
  if (!rerun) L->launches++;
  mark(L, 1, st);   // (stage 1, the scan, has no launch of its own: it runs in the permute kernel, or for very large
                    // grids and swapmoe_route_static in the router's last CTA)

  // Permute CTAs: every row group of a token tile gets its own CTA.  About 1.5 CTAs per SM, more when the rows are
  // long (at most 96 KB of rows per CTA).  Not more than that: the grouped GEMM's CTAs can only be launched into the
  // SMs the permute CTAs have left, and launching that grid takes 3-4 us once it can start (8192 tokens of
  // d_model 768: three groups 137.7 us per forward, two groups 135.3).
  int groups_planned = (3 * L->sm_count / 2 + n_cta - 1) / n_cta;
  {
    const long long row_bytes = (long long)n_pairs * c.d_model * L->elem;
    const int by_bytes = (int)((row_bytes + (long long)n_cta * (96 << 10) - 1) / ((long long)n_cta * (96 << 10)));
    if (by_bytes > groups_planned) groups_planned = by_bytes;
    const int max_groups = (tok_tile * c.top_k + 7) / 8;
    if (L->permute_groups > 0) groups_planned = L->permute_groups;
    if (groups_planned > max_groups) groups_planned = max_groups;
    if (groups_planned < 1) groups_planned = 1;
  }
  PermuteArgs pa;
  pa.x = x; pa.slot = L->slot; pa.cta_base = L->cta_base; pa.offset = L->offset;
  pa.pad_offset = L->pad_offset; pa.perm = L->perm; pa.inv = L->inv; pa.inv_pad = L->inv_pad;
  pa.row_pair = L->row_pair;
  pa.xp = L->xp; pa.T = T; pa.d = c.d_model; pa.k = c.top_k; pa.K = c.K; pa.tok_tile = tok_tile;
  pa.own_scan = own_scan ? 1 : 0;
  pa.scan = sa;
  mark(L, 2, st);
  const int groups = groups_planned;
  // own_scan: three extra columns of CTAs, whose first CTAs reduce the three per-expert scores
  if (!rerun) {
    if (launch_kernel(permute_gather_kernel<DT>, dim3(n_cta + (own_scan ? 3 : 0), groups), dim3(kPermThreads), 0, st, pdl,
                      pa) != cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    L->launches++;
  }
  mark(L, 3, st);
  bool combined = false;
  int y_split = 1;
  if (use_tc) {
    cudaEvent_t mid = L->stage_events ? static_cast<cudaEvent_t>(L->stage_events[4]) : nullptr;
    int32_t rc;
    L->tc.only = rerun;
    if (L->small_path && n_pairs <= 64 && c.act == SWAPMOE_ACT_RELU) {
      if (rerun) return SWAPMOE_ERR_UNSUPPORTED;
      rc = tc_ffn_small(L->tc, L->small, c, L->xp, L->h, L->y, out, L->rows_pad_max, L->arena_in, L->arena_out,
                        L->tiles, L->n_tiles, L->row_pair, L->mgate, max_tiles, T, L->status, st, pdl,
                        &L->launches, &combined, mid);
    } else if (mt == 2 && L->gemm_pairs > 0 && c.d_ff % 256 == 0) {
      // 256-row tiles: GEMM-1 always on CTA pairs (its one-CTA form pulls 48 KB per k-block); GEMM-2 on pairs for
      // very large slots, else on one CTA with two row sub-tiles (same bytes per flop, and a tile whose second
      // half is empty costs half; cfg3: 128.6 -> 126.8 us)
      rc = tc_ffn_pair(L->tc, L->gemm_pairs, c, L->h, L->y, out, L->tiles, L->n_tiles, L->row_pair, L->mgate, max_tiles,
                       T, L->status, st, pdl, &L->launches, &combined, mid, use_pairs, L->row_group);
    } else {
      rc = tc_ffn(L->tc, c, L->h, L->y, out, L->tiles, L->n_tiles, L->tiles_b, L->n_tiles_b, L->row_pair, L->mgate,
                  max_tiles, mt, T,
                  L->status, st, pdl, &L->launches, &combined, mid, L->row_group);
    }
    L->tc.only = 0;
    if (rc != SWAPMOE_OK) return rc;
  } else if (use_tc32) {
    cudaEvent_t mid = L->stage_events ? static_cast<cudaEvent_t>(L->stage_events[4]) : nullptr;
    L->tc32.only = rerun;
    const int32_t rc = tc_ffn_f32(L->tc32, c, L->h, L->y, (long long)L->rows_pad_max * c.d_model, L->y_copies, L->tiles,
                                  L->n_tiles, max_tiles, T, L->status, st, pdl, &L->launches, &y_split, mid, swap32);
    L->tc32.only = 0;
    if (rc != SWAPMOE_OK) return rc;
  } else {
    if (rerun) return SWAPMOE_ERR_UNSUPPORTED;
    MmaGemmArgs g1;
    g1.A = L->xp; g1.W = L->arena_in; g1.C = L->h; g1.tiles = L->tiles; g1.n_tiles = L->n_tiles;
    g1.slot_stride = (long long)L->nin * c.d_ff * c.d_model;
    g1.gate_offset = (long long)c.d_ff * c.d_model;
    g1.N = c.d_ff; g1.Kdim = c.d_model; g1.split_stride = 0;
    const dim3 grid1(c.d_ff / kMmaBN, max_tiles);
    const cudaError_t e =
        c.act == SWAPMOE_ACT_SWIGLU
            ? launch_kernel(gemm_tf32x3_kernel<DT, DT, DT, kEpiSwiglu>, grid1, dim3(kMmaThreads), 0, st, pdl, g1)
            : launch_kernel(gemm_tf32x3_kernel<DT, DT, DT, kEpiRelu>, grid1, dim3(kMmaThreads), 0, st, pdl, g1);
    if (e != cudaSuccess) return SWAPMOE_ERR_CUDA;
    L->launches++;
    mark(L, 4, st);
    MmaGemmArgs g2;
    g2.A = L->h; g2.W = L->arena_out; g2.C = L->y; g2.tiles = L->tiles; g2.n_tiles = L->n_tiles;
    g2.slot_stride = (long long)c.d_ff * c.d_model;
    g2.gate_offset = 0;
    g2.N = c.d_model; g2.Kdim = c.d_ff;
    // Few output tiles and a long contraction: slice the contraction so that every SM has work.
    // The slices land in separate copies of y and the combine kernel adds them in order.
    const long long tiles_est = ((long long)n_pairs / kMmaBM + (n_pairs < c.K ? n_pairs : c.K) / 2 + 1) *
                                (c.d_model / kMmaBN);
    y_split = mma_pick_split(tiles_est, L->sm_count, c.d_ff, L->y_copies);
    g2.split_stride = (long long)L->rows_pad_max * c.d_model;
    const dim3 grid2(c.d_model / kMmaBN, max_tiles, y_split);
    if (launch_kernel(gemm_tf32x3_kernel<DT, DT, float, kEpiNone>, grid2, dim3(kMmaThreads), 0, st, pdl, g2) !=
        cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    L->launches++;
  }

  CombineArgs ca;
  ca.y = L->y; ca.inv_pad = L->inv_pad; ca.mgate = L->mgate; ca.out = out;
  ca.T = T; ca.d = c.d_model; ca.k = c.top_k;
  ca.n_split = y_split; ca.split_stride = (long long)L->rows_pad_max * c.d_model;
  const long long work = (long long)T * (c.d_model / 8);
  mark(L, 5, st);
  if (rerun) return check_launch();      // neither the combine kernel nor the taps' validity change
  if (!combined) {
    if (launch_kernel(combine_kernel<DT>, dim3((unsigned)((work + 255) / 256)), dim3(256), 0, st, pdl, ca) !=
        cudaSuccess)
      return SWAPMOE_ERR_CUDA;
    L->launches++;
  }
  mark(L, 6, st);
  // what the debug taps may read back: h unless the small-batch kernels kept it on chip, y when GEMM-2 wrote it
  L->h_valid = true;
  L->y_valid = !combined;
  L->y_split_last = y_split;
  return check_launch();
}

int32_t forward_checked(swapmoe_layer* L, const void* x, const float* ext, void* out, int32_t T,
                        void* stream) {
  if (!L || T < 0) return SWAPMOE_ERR_INVALID_ARG;
  if (T == 0) { L->last_T = 0; return SWAPMOE_OK; }
  if (!x || !out) return SWAPMOE_ERR_INVALID_ARG;
  if (!L->router_set || !L->resident_set) return SWAPMOE_ERR_NOT_READY;
  if (T > L->cfg.max_tokens) return SWAPMOE_ERR_TOO_MANY_TOKENS;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(out)) & 15) return SWAPMOE_ERR_INVALID_ARG;
  L->last_T = T;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (L->cfg.dtype == SWAPMOE_BF16) return forward_impl<bf16>(L, x, ext, out, T, st);
  return forward_impl<float>(L, x, ext, out, T, st);
}

// H / Y taps: the hidden activations and the expert outputs live in the padded workspace (slot
// segments start at multiples of 128 rows); the tap delivers the T*k occupied rows in position
// order (row `pos` belongs to pair perm[pos]), one copy per slot segment.
int32_t debug_copy_rows(swapmoe_layer* L, int32_t which, void* host, size_t bytes, cudaStream_t st) {
  const swapmoe_config_t& c = L->cfg;
  const size_t P = (size_t)L->last_T * c.top_k;
  const bool is_h = which == SWAPMOE_TAP_H;
  if (is_h ? !L->h_valid : (!L->y_valid || L->y_split_last != 1)) return SWAPMOE_ERR_UNSUPPORTED;
  const size_t row_bytes = is_h ? (size_t)c.d_ff * L->elem : (size_t)c.d_model * sizeof(float);
  if (bytes != P * row_bytes) return SWAPMOE_ERR_INVALID_ARG;
  if (P == 0) return SWAPMOE_OK;
  int32_t count[kMaxSlots], pad[kMaxSlots + 1];
  if (!cuda_ok(cudaMemcpyAsync(count, L->count, sizeof(int32_t) * c.K, cudaMemcpyDeviceToHost, st)) ||
      !cuda_ok(cudaMemcpyAsync(pad, L->pad_offset, sizeof(int32_t) * (c.K + 1), cudaMemcpyDeviceToHost, st)) ||
      !cuda_ok(cudaStreamSynchronize(st)))
    return SWAPMOE_ERR_CUDA;
  const char* base = is_h ? static_cast<const char*>(L->h) : reinterpret_cast<const char*>(L->y);
  char* dst = static_cast<char*>(host);
  for (int s = 0; s < c.K; ++s) {
    if (count[s] == 0) continue;
    if (!cuda_ok(cudaMemcpyAsync(dst, base + (size_t)pad[s] * row_bytes, (size_t)count[s] * row_bytes,
                                 cudaMemcpyDeviceToHost, st)))
      return SWAPMOE_ERR_CUDA;
    dst += (size_t)count[s] * row_bytes;
  }
  return cuda_ok(cudaStreamSynchronize(st)) ? SWAPMOE_OK : SWAPMOE_ERR_CUDA;
}

}  // namespace

extern "C" {

int32_t swapmoe_create(swapmoe_layer_t** out, const swapmoe_config_t* cfg) {
  if (!out || !cfg) return SWAPMOE_ERR_INVALID_ARG;
  const swapmoe_config_t c = *cfg;
  if (c.E < 1 || c.K < 1 || c.top_k < 1 || c.d_model < 1 || c.d_ff < 1 || c.max_tokens < 1 ||
      c.spare_slots < 0)
    return SWAPMOE_ERR_INVALID_ARG;
  if (c.K < c.top_k || c.K > c.E) return SWAPMOE_ERR_INVALID_ARG;
  if (c.dtype != SWAPMOE_F32 && c.dtype != SWAPMOE_BF16) return SWAPMOE_ERR_INVALID_ARG;
  if (c.act != SWAPMOE_ACT_RELU && c.act != SWAPMOE_ACT_SWIGLU) return SWAPMOE_ERR_INVALID_ARG;
  if (c.renorm_topk != 0 && c.renorm_topk != 1) return SWAPMOE_ERR_INVALID_ARG;
  if (c.E > kMaxE || c.K + c.spare_slots > kMaxSlots || c.top_k > kMaxTopK) return SWAPMOE_ERR_UNSUPPORTED;
  if (c.d_model % 64 || c.d_ff % 64) return SWAPMOE_ERR_UNSUPPORTED;
  if ((long long)c.max_tokens * c.top_k >= (1ll << 24)) return SWAPMOE_ERR_UNSUPPORTED;

  int dev = 0;
  if (!cuda_ok(cudaGetDevice(&dev))) { cudaGetLastError(); return SWAPMOE_ERR_CUDA; }
  cudaDeviceProp prop;
  if (!cuda_ok(cudaGetDeviceProperties(&prop, dev))) { cudaGetLastError(); return SWAPMOE_ERR_CUDA; }
  if (prop.major != 10) return SWAPMOE_ERR_UNSUPPORTED;  // kernels are built for sm_100a only

  swapmoe_layer* L = new (std::nothrow) swapmoe_layer();
  if (!L) return SWAPMOE_ERR_NO_MEMORY;
  std::memset(L, 0, sizeof(*L));
  L->cfg = c;
  L->device = dev;
  L->sm_count = prop.multiProcessorCount;
  {
    const char* env = std::getenv("SWAPMOE_PDL");      // SWAPMOE_PDL=0 launches every kernel fully serialised
    L->use_pdl = !(env && env[0] == '0');
    env = std::getenv("SWAPMOE_PERMUTE_GROUPS");        // CTAs per token tile of the permute kernel (0: automatic)
    L->permute_groups = env ? std::atoi(env) : 0;
    env = std::getenv("SWAPMOE_ROUTER_TOK");            // force the router's token tile (32, 64 or 128)
    L->router_tok = env ? std::atoi(env) : 0;
    if (L->router_tok != 32 && L->router_tok != 64 && L->router_tok != 128) L->router_tok = 0;
    env = std::getenv("SWAPMOE_SMALL_PATH");            // SWAPMOE_SMALL_PATH=0: general GEMM kernels for small batches too
    L->small_path = !(env && env[0] == '0');
    env = std::getenv("SWAPMOE_ROW_GROUP");             // row tiles per scheduling group of the grouped GEMMs
    L->row_group = env && std::atoi(env) > 0 ? std::atoi(env) : 0;
    // L2 weight prefetch from the router's idle blocks (SWAPMOE_PREFETCH_MB=<MB> switches it on).  Off by default:
    // since the slot scan left the router, the router is too short to hide it - every megabyte prefetched slows
    // the router by about as much as it speeds GEMM-1 up (B200, 2048 tokens: 0 / 24 / 56 MB -> 54.7 / 54.9 / 56.4 us).
    env = std::getenv("SWAPMOE_PREFETCH_MB");
    L->l2_prefetch_bytes = env ? std::atoll(env) << 20 : 0;
    L->prefetch = L->l2_prefetch_bytes > 0;
    env = std::getenv("SWAPMOE_FP32_SWAP");             // SWAPMOE_FP32_SWAP=0: fp32 layers always on 128-token tiles
    L->fp32_swap = !(env && env[0] == '0');
    env = std::getenv("SWAPMOE_PREFETCH_MIN_PAIRS");
    L->prefetch_min_pairs = env ? std::max(1, std::atoi(env)) : 1;
  }
  L->nin = c.act == SWAPMOE_ACT_SWIGLU ? 2 : 1;
  L->elem = c.dtype == SWAPMOE_BF16 ? 2 : 4;

  const size_t T = (size_t)c.max_tokens, P = T * c.top_k;
  // router CTAs: 32-token tiles at least; batches of up to 64 tokens may use eight-token tiles
  size_t n_cta = (T + kTokTile - 1) / kTokTile;
  {
    const size_t small = std::min<size_t>((T + kRsTok - 1) / kRsTok, kRsMaxTokens / kRsTok);
    if (small > n_cta) n_cta = small;
    const size_t mid = std::min<size_t>((T + 2 * kRsTok - 1) / (2 * kRsTok), 256);   // sixteen-token CTAs
    if (mid > n_cta) n_cta = mid;
    const size_t f32small = std::min<size_t>((T + kRsTok - 1) / kRsTok, 256);         // fp32: eight-token CTAs, one wave
    if (c.dtype == SWAPMOE_F32 && f32small > n_cta) n_cta = f32small;
  }
  const size_t rows_pad = align_up(P + (size_t)c.K * kSegAlign, kSegAlign);
  const size_t max_tiles = (P + kMmaBM - 1) / kMmaBM + c.K;
  L->rows_pad_max = (int32_t)rows_pad;

  Carver cv;
  const size_t o_logits = cv.take<float>(T * c.E);
  const size_t o_ugate = cv.take<float>(P), o_mgate = cv.take<float>(P), o_xnorm = cv.take<float>(T);
  const size_t o_cta_imp = cv.take<float>(n_cta * c.E);
  const size_t o_cta_cnt = cv.take<float>(n_cta * c.E), o_cta_mimp = cv.take<float>(n_cta * c.K);
  const size_t o_cnt = cv.take<float>(c.E), o_mimp = cv.take<float>(c.E);
  const size_t o_imp = cv.take<float>(c.E), o_enorm = cv.take<float>(c.E);
  const size_t o_uidx = cv.take<int32_t>(P), o_midx = cv.take<int32_t>(P), o_slot = cv.take<int32_t>(P);
  const size_t o_cta_hist = cv.take<int32_t>(n_cta * c.K), o_cta_base = cv.take<int32_t>(n_cta * c.K);
  const size_t o_count = cv.take<int32_t>(c.K), o_offset = cv.take<int32_t>(c.K + 1);
  const size_t o_pad = cv.take<int32_t>(c.K + 1);
  const size_t o_perm = cv.take<int32_t>(P), o_inv = cv.take<int32_t>(P), o_invp = cv.take<int32_t>(P);
  const size_t o_rowpair = cv.take<int32_t>(rows_pad);
  const size_t o_ntiles = cv.take<int32_t>(4), o_e2s = cv.take<int32_t>(c.E);
  const size_t o_phys = cv.take<int32_t>(kMaxSlots), o_s2e = cv.take<int32_t>(kMaxSlots);
  const size_t o_status = cv.take<int32_t>(4);
  const size_t o_ticket = cv.take<unsigned>(4);
  const size_t o_touched = cv.take<unsigned long long>(2);
  const size_t o_dec_stats = cv.take<unsigned long long>(2), o_dec_recent = cv.take<int32_t>(kDecRecent);
  // (at least 32 entries each: the grouped GEMM's producer warp fetches the first 32 descriptors in one go)
  const size_t o_tiles = cv.take<TileDesc>(max_tiles < 32 ? 32 : max_tiles);
  const size_t o_tiles_b = cv.take<TileDesc>(max_tiles < 32 ? 32 : max_tiles), o_ntiles_b = cv.take<int32_t>(4);
  const size_t o_xp = cv.take<char>(rows_pad * c.d_model * L->elem);
  const size_t o_h = cv.take<char>(rows_pad * c.d_ff * L->elem);
  // up to four copies of y for a sliced contraction in the CUDA-core GEMM-2, when they stay small
  L->y_copies = (rows_pad * c.d_model * sizeof(float) * 4 <= (size_t)(64u << 20)) ? 4 : 1;
  const size_t o_y = cv.take<float>(rows_pad * c.d_model * L->y_copies);
  const size_t o_xs = cv.take<char>(T * c.d_model * L->elem);
  const size_t o_os = cv.take<char>(T * c.d_model * L->elem);
  {
    // Measured on B200 (d_model 1024, d_ff 4096, top-1), us per layer for 1 .. 6 tokens: the one-launch path 18.6 /
    // 23.5 / 29.7 / 33.8 / 38.2 / 42.7, the general kernels 30.5 / 31.8 / 33.0 / 34.1 / 39.2 / 40.5: it wins up to
    // five pairs.
    L->decode_max_pairs = 5;
    const char* envt = std::getenv("SWAPMOE_DECODE_MAX_PAIRS");  // 1..32: use the one-launch path up to this many pairs
    if (envt && std::atoi(envt) >= 1 && std::atoi(envt) <= kDecMaxPairs) L->decode_max_pairs = std::atoi(envt);
    const char* env = std::getenv("SWAPMOE_DECODE_PATH");   // SWAPMOE_DECODE_PATH=0: general kernels for tiny batches too
    L->decode_path = c.dtype == SWAPMOE_BF16 && !(env && env[0] == '0') &&
                     decode_smem_bytes(c.d_model) <= (size_t)(226 << 10) &&
                     decode_ws_floats(c.d_model, c.d_ff, c.top_k) * sizeof(float) <= ((size_t)64 << 20);
  }
  const size_t o_dec_ws = cv.take<float>(L->decode_path ? decode_ws_floats(c.d_model, c.d_ff, c.top_k) : 1);
  const size_t o_dec_tk = cv.take<unsigned>(L->decode_path ? decode_ticket_count(c.d_ff, c.K) : 1);
  L->ws_bytes = cv.off;
  if (!cuda_ok(cudaMalloc(&L->ws_base, L->ws_bytes))) { cudaGetLastError(); delete L; return SWAPMOE_ERR_NO_MEMORY; }
  char* b = L->ws_base;
  L->logits = (float*)(b + o_logits); L->ugate = (float*)(b + o_ugate); L->mgate = (float*)(b + o_mgate);
  L->xnorm = (float*)(b + o_xnorm); L->cta_imp = (float*)(b + o_cta_imp); L->imp = (float*)(b + o_imp);
  L->cta_cnt = (float*)(b + o_cta_cnt); L->cta_mimp = (float*)(b + o_cta_mimp);
  L->cnt = (float*)(b + o_cnt); L->mimp = (float*)(b + o_mimp);
  L->enorm = (float*)(b + o_enorm); L->uidx = (int32_t*)(b + o_uidx); L->midx = (int32_t*)(b + o_midx);
  L->slot = (int32_t*)(b + o_slot); L->cta_hist = (int32_t*)(b + o_cta_hist);
  L->cta_base = (int32_t*)(b + o_cta_base); L->count = (int32_t*)(b + o_count);
  L->offset = (int32_t*)(b + o_offset); L->pad_offset = (int32_t*)(b + o_pad);
  L->perm = (int32_t*)(b + o_perm); L->inv = (int32_t*)(b + o_inv); L->inv_pad = (int32_t*)(b + o_invp);
  L->row_pair = (int32_t*)(b + o_rowpair);
  L->n_tiles = (int32_t*)(b + o_ntiles); L->e2s = (int32_t*)(b + o_e2s); L->phys = (int32_t*)(b + o_phys);
  L->s2e = (int32_t*)(b + o_s2e); L->status = (int32_t*)(b + o_status);
  L->ticket = (unsigned*)(b + o_ticket);
  L->touched = (unsigned long long*)(b + o_touched);
  L->dec_pf_stats = (unsigned long long*)(b + o_dec_stats); L->dec_recent = (int32_t*)(b + o_dec_recent);
  L->tiles = (TileDesc*)(b + o_tiles);
  L->tiles_b = (TileDesc*)(b + o_tiles_b); L->n_tiles_b = (int32_t*)(b + o_ntiles_b);
  L->xp = b + o_xp; L->h = b + o_h; L->y = (float*)(b + o_y);
  L->x_stage = b + o_xs; L->out_stage = b + o_os;
  L->dec_ws = (float*)(b + o_dec_ws); L->dec_tickets = (unsigned*)(b + o_dec_tk);

  bool ok = cuda_ok(cudaMemset(L->imp, 0, sizeof(float) * c.E));
  ok = ok && cuda_ok(cudaMemset(L->cnt, 0, sizeof(float) * c.E));
  ok = ok && cuda_ok(cudaMemset(L->mimp, 0, sizeof(float) * c.E));
  ok = ok && cuda_ok(cudaMemset(L->status, 0, sizeof(int32_t) * 4));
  ok = ok && cuda_ok(cudaMemset(L->ticket, 0, sizeof(unsigned) * 4));
  ok = ok && cuda_ok(cudaMemset(L->touched, 0, sizeof(unsigned long long) * 2));
  ok = ok && cuda_ok(cudaMemset(L->dec_pf_stats, 0, sizeof(unsigned long long) * 2));
  ok = ok && cuda_ok(cudaMemset(L->dec_recent, 0xff, sizeof(int32_t) * kDecRecent));      // -1: nothing served yet
  {
    // Decode steps: L2 prefetch of the experts the layer served last (activation locality, Section 2.2).  Off by
    // default: measured on B200 with the synthetic decode traffic (a token keeps its expert of the step before in
    // 11 % of the steps, one of the last three in 29 %) the step got no faster (18.3 -> 18.6 .. 19.2 us per layer at one
    // token per step): even a correct guess saves little, because the step is bound by its chain of dependent
    // phases, not by the 2.6 us its weights take from HBM.
    const char* envp = std::getenv("SWAPMOE_DECODE_PREFETCH");   // 0 .. 4 recently served experts
    L->dec_pf_depth = envp ? std::min(std::max(std::atoi(envp), 0), kDecRecent) : 0;
  }
  if (L->decode_path) {
    ok = ok && cuda_ok(cudaMemset(L->dec_tickets, 0, sizeof(unsigned) * decode_ticket_count(c.d_ff, c.K)));
    ok = ok && cuda_ok(decode_fused_set_smem_limit((int)decode_smem_bytes(c.d_model)));
  }
  ok = ok && cuda_ok(cudaFuncSetAttribute(router_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          226 * 1024));
  // Rows of the padded workspaces that no pair occupies are computed on but never
  // read back; start them at zero so they hold finite values.
  ok = ok && cuda_ok(cudaMemset(L->xp, 0, rows_pad * c.d_model * L->elem));
  ok = ok && cuda_ok(router_gate_set_smem_limit<float>()) && cuda_ok(router_gate_set_smem_limit<bf16>());
  ok = ok && tc_init(L->tc, c, L->xp, L->h, L->y, L->rows_pad_max) == SWAPMOE_OK;
  L->tc32.enabled = L->tc32.arena_bound = false;
  L->encode32 = nullptr;
  {
    const char* env = std::getenv("SWAPMOE_FP32_TC");        // SWAPMOE_FP32_TC=0: warp-level mma (or FFMA) for fp32 layers
    if (ok && c.dtype == SWAPMOE_F32 && !(env && env[0] == '0')) {
      L->encode32 = tc_get_encoder();
      ok = tc_f32_init(L->tc32, L->encode32, c, L->xp, L->h, L->rows_pad_max, L->sm_count) == SWAPMOE_OK;
    }
  }
  if (L->tc.encode == nullptr) L->decode_path = false;     // its W_out loads need a tensor map
  {
    const char* env = std::getenv("SWAPMOE_PAIR_GEMM");      // SWAPMOE_PAIR_GEMM=0: one CTA per tile for every shape
    L->gemm_pairs = (ok && L->tc.enabled && !(env && env[0] == '0')) ? tc_pair_init(L->sm_count) : 0;
    env = std::getenv("SWAPMOE_PAIR_MIN_ROWS");
    L->pair_min_rows = env ? std::max(160, std::atoi(env)) : 1024;
    if (std::getenv("SWAPMOE_DEBUG")) std::fprintf(stderr, "swapmoe: gemm_pairs=%d\n", L->gemm_pairs);
  }
  {
    const char* env = std::getenv("SWAPMOE_SMALL_ROUTER");   // SWAPMOE_SMALL_ROUTER=0: tcgen05 router for small batches too
    L->small_router = c.dtype == SWAPMOE_BF16 && !(env && env[0] == '0') &&
                      router_small_smem_bytes(c.d_model, 1) <= (size_t)(226 << 10);
    if (L->small_router)
      ok = ok && cuda_ok(cudaFuncSetAttribute(router_small_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)router_small_smem_bytes(c.d_model, 1)));
    L->small_router_f32 = c.dtype == SWAPMOE_F32 && !(env && env[0] == '0') &&
                          router_small_f32_smem_bytes(c.d_model) <= (size_t)(226 << 10);
    if (L->small_router_f32)
      ok = ok && cuda_ok(cudaFuncSetAttribute(router_small_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)router_small_f32_smem_bytes(c.d_model)));
    // sixteen-token CTAs: while the grid stays within one wave of CTAs and the shared memory fits
    L->small_router_max_t = 0;
    if (L->small_router && router_small_smem_bytes(c.d_model, 2) <= (size_t)(226 << 10)) {
      L->small_router_max_t = 2 * kRsTok * L->sm_count;
      const char* envm = std::getenv("SWAPMOE_SMALL_ROUTER_MAX_T");
      if (envm) L->small_router_max_t = std::min(std::atoi(envm), 2 * kRsTok * 256);
      ok = ok && cuda_ok(cudaFuncSetAttribute(router_small_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)router_small_smem_bytes(c.d_model, 2)));
    }
  }
  if (ok && L->tc.enabled) ok = tc_small_set_attrs();
  ok = ok && cuda_ok(cudaStreamCreateWithFlags(&L->s_in, cudaStreamNonBlocking));
  ok = ok && cuda_ok(cudaStreamCreateWithFlags(&L->s_out, cudaStreamNonBlocking));
  ok = ok && cuda_ok(cudaEventCreateWithFlags(&L->ev_in, cudaEventDisableTiming));
  ok = ok && cuda_ok(cudaEventCreateWithFlags(&L->ev_comp, cudaEventDisableTiming));
  ok = ok && cuda_ok(cudaEventCreateWithFlags(&L->ev_out, cudaEventDisableTiming));
  ok = ok && cuda_ok(cudaEventCreateWithFlags(&L->ev_load, cudaEventDisableTiming));
  if (!ok) { cudaGetLastError(); swapmoe_destroy(L); return SWAPMOE_ERR_CUDA; }   // frees whatever was created
  *out = L;
  return SWAPMOE_OK;
}

int32_t swapmoe_destroy(swapmoe_layer_t* L) {
  if (!L) return SWAPMOE_OK;
  if (L->s_in) cudaStreamDestroy(L->s_in);
  if (L->s_out) cudaStreamDestroy(L->s_out);
  if (L->ev_in) cudaEventDestroy(L->ev_in);
  if (L->ev_comp) cudaEventDestroy(L->ev_comp);
  if (L->ev_out) cudaEventDestroy(L->ev_out);
  if (L->ev_load) cudaEventDestroy(L->ev_load);
  cudaFree(L->ws_base);
  delete L;
  return SWAPMOE_OK;
}

int32_t swapmoe_set_router(swapmoe_layer_t* L, const void* Wr_dev, const float* enorm_host, void* stream) {
  if (!L || !Wr_dev || !enorm_host) return SWAPMOE_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(Wr_dev) & 15) return SWAPMOE_ERR_INVALID_ARG;
  EnormTable t;
  std::memset(&t, 0, sizeof(t));
  for (int i = 0; i < L->cfg.E; ++i) t.v[i] = enorm_host[i];
  if (L->tc.router_ok &&
      !tc_encode_2d(L->tc.encode, &L->tc.map_wr, Wr_dev, (uint64_t)L->cfg.E, (uint64_t)L->cfg.d_model,
                    (uint32_t)router_tc_epad(L->cfg.E)))
    return SWAPMOE_ERR_CUDA;
  set_enorm_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(t, L->cfg.E, L->enorm);
  L->launches++;
  L->Wr = Wr_dev;
  L->router_set = true;
  return check_launch();
}

int32_t swapmoe_set_resident(swapmoe_layer_t* L, const int32_t* s2e, const int32_t* phys,
                             const void* arena_in, const void* arena_out, void* stream) {
  if (!L || !s2e || !arena_in || !arena_out) return SWAPMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(arena_in) | reinterpret_cast<uintptr_t>(arena_out)) & 15)
    return SWAPMOE_ERR_INVALID_ARG;
  const swapmoe_config_t& c = L->cfg;
  const int P = c.K + c.spare_slots;
  SlotTables t;
  for (int e = 0; e < kMaxE; ++e) t.e2s[e] = -1;
  bool used[kMaxSlots];
  for (int p = 0; p < kMaxSlots; ++p) { used[p] = false; t.phys[p] = 0; t.s2e[p] = -1; }
  for (int s = 0; s < c.K; ++s) {
    const int e = s2e[s];
    if (e < 0 || e >= c.E || t.e2s[e] != -1) return SWAPMOE_ERR_BAD_SLOT_TABLE;
    t.e2s[e] = s;
    t.s2e[s] = e;
    const int p = phys ? phys[s] : s;
    if (p < 0 || p >= P || used[p]) return SWAPMOE_ERR_BAD_SLOT_TABLE;
    used[p] = true;
    t.phys[s] = p;
  }
  if (arena_in != L->arena_in || arena_out != L->arena_out) {
    L->small.valid = false;
    int32_t rc = tc_bind_arena(L->tc, c, arena_in, arena_out);
    if (rc != SWAPMOE_OK) return rc;
    rc = tc_f32_bind_arena(L->tc32, L->encode32, c, arena_in, arena_out);
    if (rc != SWAPMOE_OK) return rc;
    // column slices of W_out for the one-launch decode kernel: 32 columns x 256 rows, 64-byte swizzle
    if (L->decode_path &&
        !tc_encode_2d_box(L->tc.encode, &L->dec_map_wo, arena_out, (uint64_t)P * c.d_model, (uint64_t)c.d_ff,
                          (uint32_t)kDecJB, (uint32_t)kDecOutRows, CU_TENSOR_MAP_SWIZZLE_64B))
      return SWAPMOE_ERR_CUDA;
  }
  set_tables_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(t, c.E, c.K, L->e2s, L->phys, L->s2e);
  L->launches++;
  for (int s = 0; s < c.K; ++s) { L->h_s2e[s] = t.s2e[s]; L->h_phys[s] = t.phys[s]; }
  L->arena_in = arena_in;
  L->arena_out = arena_out;
  L->resident_set = true;
  return check_launch();
}

int32_t swapmoe_forward(swapmoe_layer_t* L, const void* x, void* out, int32_t T, void* stream) {
  return forward_checked(L, x, nullptr, out, T, stream);
}

int32_t swapmoe_forward_timed(swapmoe_layer_t* L, const void* x, void* out, int32_t T, void* stream,
                              void* const* events) {
  if (!L || !events) return SWAPMOE_ERR_INVALID_ARG;
  for (int i = 0; i < SWAPMOE_N_STAGES + 1; ++i)
    if (!events[i]) return SWAPMOE_ERR_INVALID_ARG;
  L->stage_events = events;
  const int32_t rc = forward_checked(L, x, nullptr, out, T, stream);
  L->stage_events = nullptr;
  return rc;
}

int32_t swapmoe_debug_rerun_gemm(swapmoe_layer_t* L, void* out, int32_t which, void* stream) {
  if (!L || !out || (which != 1 && which != 2)) return SWAPMOE_ERR_INVALID_ARG;
  if (L->last_T <= 0) return SWAPMOE_ERR_NOT_READY;
  L->rerun_gemm = which;
  const int32_t rc = forward_checked(L, out, nullptr, out, L->last_T, stream);   // x is not read: no router, no permute
  L->rerun_gemm = 0;
  return rc;
}

int32_t swapmoe_forward_from_logits(swapmoe_layer_t* L, const void* x, const float* logits, void* out,
                                    int32_t T, void* stream) {
  if (!logits && T > 0) return SWAPMOE_ERR_INVALID_ARG;
  return forward_checked(L, x, logits, out, T, stream);
}

int32_t swapmoe_forward_host(swapmoe_layer_t* L, const void* x_host, void* out_host, int32_t T,
                             void* stream) {
  if (!L || T < 0) return SWAPMOE_ERR_INVALID_ARG;
  if (T == 0) return SWAPMOE_OK;
  if (!x_host || !out_host) return SWAPMOE_ERR_INVALID_ARG;
  if (T > L->cfg.max_tokens) return SWAPMOE_ERR_TOO_MANY_TOKENS;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)T * L->cfg.d_model * L->elem;
  // the staging buffers are shared with the pipelined entry point: wait for its last forward (which
  // reads x_stage) and its last copy-out (which reads out_stage); no-ops when it was never used
  if (!cuda_ok(cudaStreamWaitEvent(st, L->ev_comp, 0)) || !cuda_ok(cudaStreamWaitEvent(st, L->ev_out, 0)))
    return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaMemcpyAsync(L->x_stage, x_host, bytes, cudaMemcpyHostToDevice, st))) return SWAPMOE_ERR_CUDA;
  const int32_t rc = forward_checked(L, L->x_stage, nullptr, L->out_stage, T, stream);
  if (rc != SWAPMOE_OK) return rc;
  if (!cuda_ok(cudaMemcpyAsync(out_host, L->out_stage, bytes, cudaMemcpyDeviceToHost, st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  return SWAPMOE_OK;
}

int32_t swapmoe_forward_host_async(swapmoe_layer_t* L, const void* x_host, void* out_host, int32_t T,
                                   void* stream) {
  if (!L || T < 0) return SWAPMOE_ERR_INVALID_ARG;
  if (T == 0) return SWAPMOE_OK;
  if (!x_host || !out_host) return SWAPMOE_ERR_INVALID_ARG;
  if (T > L->cfg.max_tokens) return SWAPMOE_ERR_TOO_MANY_TOKENS;
  if (!L->router_set || !L->resident_set) return SWAPMOE_ERR_NOT_READY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)T * L->cfg.d_model * L->elem;
  // copy-in stream: the staging buffer is free once the previous forward of this layer has run
  bool ok = cuda_ok(cudaStreamWaitEvent(L->s_in, L->ev_comp, 0));
  ok = ok && cuda_ok(cudaMemcpyAsync(L->x_stage, x_host, bytes, cudaMemcpyHostToDevice, L->s_in));
  ok = ok && cuda_ok(cudaEventRecord(L->ev_in, L->s_in));
  // compute stream: needs the tokens, and the output staging buffer must have been copied out
  ok = ok && cuda_ok(cudaStreamWaitEvent(st, L->ev_in, 0));
  ok = ok && cuda_ok(cudaStreamWaitEvent(st, L->ev_out, 0));
  if (!ok) return SWAPMOE_ERR_CUDA;
  const int32_t rc = forward_checked(L, L->x_stage, nullptr, L->out_stage, T, stream);
  if (rc != SWAPMOE_OK) return rc;
  ok = cuda_ok(cudaEventRecord(L->ev_comp, st));
  // copy-out stream
  ok = ok && cuda_ok(cudaStreamWaitEvent(L->s_out, L->ev_comp, 0));
  ok = ok && cuda_ok(cudaMemcpyAsync(out_host, L->out_stage, bytes, cudaMemcpyDeviceToHost, L->s_out));
  ok = ok && cuda_ok(cudaEventRecord(L->ev_out, L->s_out));
  return ok ? SWAPMOE_OK : SWAPMOE_ERR_CUDA;
}

int32_t swapmoe_host_wait(swapmoe_layer_t* L) {
  if (!L) return SWAPMOE_ERR_INVALID_ARG;
  return cuda_ok(cudaEventSynchronize(L->ev_out)) ? SWAPMOE_OK : SWAPMOE_ERR_CUDA;
}

int32_t swapmoe_read_importance_kind(swapmoe_layer_t* L, int32_t kind, float* imp_host, int32_t reset,
                                     void* stream) {
  if (!L || !imp_host) return SWAPMOE_ERR_INVALID_ARG;
  float* acc = kind == SWAPMOE_IMP_EQ1 ? L->imp : kind == SWAPMOE_IMP_COUNT ? L->cnt
             : kind == SWAPMOE_IMP_EQ1_MASKED ? L->mimp : nullptr;
  if (!acc) return SWAPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!cuda_ok(cudaMemcpyAsync(imp_host, acc, sizeof(float) * L->cfg.E, cudaMemcpyDeviceToHost, st)))
    return SWAPMOE_ERR_CUDA;
  if (reset && !cuda_ok(cudaMemsetAsync(acc, 0, sizeof(float) * L->cfg.E, st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  return SWAPMOE_OK;
}

int32_t swapmoe_read_scores_async(swapmoe_layer_t* L, int32_t kinds_mask, float* scores_host_pinned, int32_t reset,
                                  void* stream) {
  if (!L || !scores_host_pinned || kinds_mask < 1 || kinds_mask > 7) return SWAPMOE_ERR_INVALID_ARG;
  // pinned host memory is mapped into the device's address space: the kernel writes it directly
  void* dst = nullptr;
  if (!cuda_ok(cudaHostGetDevicePointer(&dst, scores_host_pinned, 0)) || !dst) { cudaGetLastError(); return SWAPMOE_ERR_INVALID_ARG; }
  ScoreSnapshot sn;
  sn.acc[0] = L->imp; sn.acc[1] = L->cnt; sn.acc[2] = L->mimp;
  sn.dst = static_cast<float*>(dst); sn.E = L->cfg.E; sn.mask = kinds_mask; sn.reset = reset;
  snapshot_scores_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(sn);
  L->launches++;
  return check_launch();
}

int32_t swapmoe_read_importance(swapmoe_layer_t* L, float* imp_host, int32_t reset, void* stream) {
  return swapmoe_read_importance_kind(L, SWAPMOE_IMP_EQ1, imp_host, reset, stream);
}

int32_t swapmoe_read_touched_slots(swapmoe_layer_t* L, int64_t* total_host, int32_t reset, void* stream) {
  if (!L || !total_host) return SWAPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned long long v = 0;
  if (!cuda_ok(cudaMemcpyAsync(&v, L->touched, sizeof(v), cudaMemcpyDeviceToHost, st))) return SWAPMOE_ERR_CUDA;
  if (reset && !cuda_ok(cudaMemsetAsync(L->touched, 0, sizeof(v), st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  *total_host = (int64_t)v;
  return SWAPMOE_OK;
}

int32_t swapmoe_read_decode_prefetch(swapmoe_layer_t* L, int64_t* hits_host, int64_t* touched_host, int32_t reset,
                                     void* stream) {
  if (!L || !hits_host || !touched_host) return SWAPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned long long v[2] = {0, 0};
  if (!cuda_ok(cudaMemcpyAsync(v, L->dec_pf_stats, sizeof(v), cudaMemcpyDeviceToHost, st))) return SWAPMOE_ERR_CUDA;
  if (reset && !cuda_ok(cudaMemsetAsync(L->dec_pf_stats, 0, sizeof(v), st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  *hits_host = (int64_t)v[0];
  *touched_host = (int64_t)v[1];
  return SWAPMOE_OK;
}

int32_t swapmoe_topk_importance(const float* imp, int32_t E, int32_t K, int32_t* out_idx) {
  if (!imp || !out_idx || E < 1 || K < 1 || K > E || E > kMaxE) return SWAPMOE_ERR_INVALID_ARG;
  bool taken[kMaxE];
  for (int e = 0; e < E; ++e) taken[e] = false;
  for (int j = 0; j < K; ++j) {
    int best = -1;
    for (int e = 0; e < E; ++e) {
      if (taken[e]) continue;
      if (best < 0 || imp[e] > imp[best]) best = e;
    }
    taken[best] = true;
    out_idx[j] = best;
  }
  return SWAPMOE_OK;
}

int32_t swapmoe_load_slot_async(swapmoe_layer_t* L, int32_t phys, const void* in_host, const void* out_host,
                                void* compute_stream, void* side_stream, void* done_event) {
  if (!L || !in_host || !out_host) return SWAPMOE_ERR_INVALID_ARG;
  if (!L->resident_set) return SWAPMOE_ERR_NOT_READY;
  const swapmoe_config_t& c = L->cfg;
  if (phys < 0 || phys >= c.K + c.spare_slots) return SWAPMOE_ERR_INVALID_ARG;
  for (int s = 0; s < c.K; ++s)
    if (L->h_phys[s] == phys) return SWAPMOE_ERR_BAD_SLOT_TABLE;
  cudaStream_t st = static_cast<cudaStream_t>(side_stream);
  // Forwards enqueued under an EARLIER table may still read entry `phys` (it is spare only in the
  // latest table), and the grouped GEMMs request weight boxes before their dependent-launch wait:
  // the copy is ordered behind everything enqueued so far on the stream the forwards run on.
  if (side_stream != compute_stream) {
    if (!cuda_ok(cudaEventRecord(L->ev_load, static_cast<cudaStream_t>(compute_stream))) ||
        !cuda_ok(cudaStreamWaitEvent(st, L->ev_load, 0)))
      return SWAPMOE_ERR_CUDA;
  }
  const size_t in_bytes = (size_t)L->nin * c.d_ff * c.d_model * L->elem;
  const size_t out_bytes = (size_t)c.d_ff * c.d_model * L->elem;
  char* din = static_cast<char*>(const_cast<void*>(L->arena_in)) + (size_t)phys * in_bytes;
  char* dout = static_cast<char*>(const_cast<void*>(L->arena_out)) + (size_t)phys * out_bytes;
  if (!cuda_ok(cudaMemcpyAsync(din, in_host, in_bytes, cudaMemcpyHostToDevice, st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaMemcpyAsync(dout, out_host, out_bytes, cudaMemcpyHostToDevice, st))) return SWAPMOE_ERR_CUDA;
  if (done_event && !cuda_ok(cudaEventRecord(static_cast<cudaEvent_t>(done_event), st))) return SWAPMOE_ERR_CUDA;
  return SWAPMOE_OK;
}

int32_t swapmoe_debug_copy(swapmoe_layer_t* L, int32_t which, void* host, size_t bytes, void* stream) {
  if (!L || !host) return SWAPMOE_ERR_INVALID_ARG;
  const swapmoe_config_t& c = L->cfg;
  const size_t T = (size_t)L->last_T, P = T * c.top_k;
  const void* src = nullptr;
  size_t need = 0;
  switch (which) {
    case SWAPMOE_TAP_LOGITS: src = L->logits; need = T * c.E * 4; break;
    case SWAPMOE_TAP_UIDX: src = L->uidx; need = P * 4; break;
    case SWAPMOE_TAP_UGATE: src = L->ugate; need = P * 4; break;
    case SWAPMOE_TAP_MIDX: src = L->midx; need = P * 4; break;
    case SWAPMOE_TAP_MGATE: src = L->mgate; need = P * 4; break;
    case SWAPMOE_TAP_SLOT: src = L->slot; need = P * 4; break;
    case SWAPMOE_TAP_COUNT: src = L->count; need = (size_t)c.K * 4; break;
    case SWAPMOE_TAP_OFFSET: src = L->offset; need = (size_t)(c.K + 1) * 4; break;
    case SWAPMOE_TAP_PERM: src = L->perm; need = P * 4; break;
    case SWAPMOE_TAP_INV: src = L->inv; need = P * 4; break;
    case SWAPMOE_TAP_XNORM: src = L->xnorm; need = T * 4; break;
    case SWAPMOE_TAP_H:
    case SWAPMOE_TAP_Y: return debug_copy_rows(L, which, host, bytes, static_cast<cudaStream_t>(stream));
    default: return SWAPMOE_ERR_INVALID_ARG;
  }
  if (bytes != need) return SWAPMOE_ERR_INVALID_ARG;
  if (need == 0) return SWAPMOE_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!cuda_ok(cudaMemcpyAsync(host, src, need, cudaMemcpyDeviceToHost, st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  return SWAPMOE_OK;
}

int32_t swapmoe_device_status(swapmoe_layer_t* L, int32_t* detail, void* stream) {
  if (!L) return SWAPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t w[4] = {0, 0, 0, 0};
  if (!cuda_ok(cudaMemcpyAsync(w, L->status, sizeof(w), cudaMemcpyDeviceToHost, st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaMemsetAsync(L->status, 0, sizeof(w), st))) return SWAPMOE_ERR_CUDA;
  if (!cuda_ok(cudaStreamSynchronize(st))) return SWAPMOE_ERR_CUDA;
  if (detail) *detail = w[1];
  return w[0] != 0 ? SWAPMOE_ERR_DEVICE_TIMEOUT : SWAPMOE_OK;
}

int32_t swapmoe_selftest_bounded_wait(swapmoe_layer_t* L, int32_t limit_ms, void* stream) {
  if (!L || limit_ms < 1 || limit_ms > 1000) return SWAPMOE_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      L->status, 99, (unsigned long long)limit_ms * 1000000ull);
  L->launches++;
  return check_launch();
}

#ifdef SWAPMOE_TRACE
// Tracing builds only: copies the kernels' %globaltimer stamps ([4 kernels][160 CTAs][16 slots] uint64) to the host.
int32_t swapmoe_debug_trace(unsigned long long* host, int32_t clear) {
  if (!host) return SWAPMOE_ERR_INVALID_ARG;
  if (!cuda_ok(cudaDeviceSynchronize()) || !cuda_ok(cudaMemcpyFromSymbol(host, swapmoe::g_trace, sizeof(swapmoe::g_trace))))
    return SWAPMOE_ERR_CUDA;
  if (clear) {
    void* p = nullptr;
    if (!cuda_ok(cudaGetSymbolAddress(&p, swapmoe::g_trace)) || !cuda_ok(cudaMemset(p, 0, sizeof(swapmoe::g_trace))))
      return SWAPMOE_ERR_CUDA;
  }
  return SWAPMOE_OK;
}
#endif

int64_t swapmoe_launch_count(const swapmoe_layer_t* L) { return L ? L->launches : 0; }
int64_t swapmoe_workspace_bytes(const swapmoe_layer_t* L) { return L ? (int64_t)L->ws_bytes : 0; }

int32_t swapmoe_set_gemm_path(swapmoe_layer_t* L, int32_t path) {
  // 0 = automatic, 1 = warp-level mma kernels (gemm_tf32x3_kernel), 2 = tcgen05 kernels
  if (!L || path < 0 || path > 2) return SWAPMOE_ERR_INVALID_ARG;
  if (path == 2 && !tc_supported(L->cfg)) return SWAPMOE_ERR_UNSUPPORTED;
  L->gemm_path = path;
  return SWAPMOE_OK;
}

const char* swapmoe_status_string(int32_t s) {
  switch (s) {
    case SWAPMOE_OK: return "ok";
    case SWAPMOE_ERR_INVALID_ARG: return "invalid argument";
    case SWAPMOE_ERR_NOT_READY: return "router or resident set not set";
    case SWAPMOE_ERR_TOO_MANY_TOKENS: return "n_tokens exceeds max_tokens";
    case SWAPMOE_ERR_BAD_SLOT_TABLE: return "bad slot table";
    case SWAPMOE_ERR_CUDA: return "CUDA error";
    case SWAPMOE_ERR_DEVICE_TIMEOUT: return "bounded device wait timed out";
    case SWAPMOE_ERR_UNSUPPORTED: return "unsupported shape or device";
    case SWAPMOE_ERR_NO_MEMORY: return "out of host or device memory";
    default: return "unknown status";
  }
}

}  // extern "C"
