/*
 * swapmoe.h - C ABI of the B200 (sm_100a) Virtual-Expert MoE-layer forward.
 *
 * The library runs ONE thing: the forward pass of a Mixture-of-Experts layer that
 * is restricted to a small resident set of experts ("Virtual Experts", SwapMoE,
 * arXiv 2308.15030, abstract and Section 3), plus the per-expert importance score
 * (Eq. 1) that decides which experts should be resident next, and the
 * asynchronous copy that brings a new expert into a spare slot (Section 3.2).
 *
 * Conventions that hold for every call
 *   - every function returns an int32 status: 0 = SWAPMOE_OK, negative = error
 *     (swapmoe_status_string() names it).  Nothing throws or aborts.
 *   - "dev" pointers are device (HBM) addresses on the layer's GPU, "host"
 *     pointers are host addresses; `stream` / `event` are cudaStream_t /
 *     cudaEvent_t passed as void* (NULL = the legacy default stream).
 *   - matrices are row-major with the contraction index innermost:
 *     x, out [n_tokens, d_model]; router Wr [E, d_model]; expert input matrices
 *     [d_ff, d_model]; expert output matrix [d_model, d_ff].  Elements are fp32
 *     (SWAPMOE_F32) or bfloat16 (SWAPMOE_BF16) as fixed at create; logits, gate
 *     values and importance are always fp32; indices are int32.
 *   - device buffers passed in must be 16-byte aligned, are owned by the caller,
 *     are never copied unless stated, and must stay valid while work that uses
 *     them is in flight.  x and out must not overlap.
 *   - a layer object may be driven from one stream at a time.
 *   - all device work is done by this library's own kernels; there is no CPU
 *     fallback.  If no usable GPU is present create() fails with
 *     SWAPMOE_ERR_CUDA.
 */
#ifndef SWAPMOE_H_
#define SWAPMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct swapmoe_layer swapmoe_layer_t; /* opaque, owned by the library */

enum { SWAPMOE_F32 = 0, SWAPMOE_BF16 = 1 };
enum { SWAPMOE_ACT_RELU = 0, SWAPMOE_ACT_SWIGLU = 1 };

enum {
  SWAPMOE_OK = 0,
  SWAPMOE_ERR_INVALID_ARG = -1,     /* null pointer, size out of range, K < top_k ...   */
  SWAPMOE_ERR_NOT_READY = -2,       /* router or resident set not set yet               */
  SWAPMOE_ERR_TOO_MANY_TOKENS = -3, /* n_tokens > max_tokens given at create            */
  SWAPMOE_ERR_BAD_SLOT_TABLE = -4,  /* expert out of range / listed twice / bad phys    */
  SWAPMOE_ERR_CUDA = -5,            /* a CUDA runtime or driver call failed             */
  SWAPMOE_ERR_DEVICE_TIMEOUT = -6,  /* a bounded in-kernel wait gave up                 */
  SWAPMOE_ERR_UNSUPPORTED = -7,     /* shape outside what the kernels are built for     */
  SWAPMOE_ERR_NO_MEMORY = -8        /* a host or device allocation failed (create only) */
};

/* Limits of this build: E <= 256, K + spare_slots <= 64, top_k <= 4,
 * d_model and d_ff multiples of 64, max_tokens * top_k < 2^24. */
typedef struct {
  int32_t E;           /* experts of the off-the-shelf layer (Section 2)                  */
  int32_t d_model;     /* token width                                                     */
  int32_t d_ff;        /* expert hidden width                                             */
  int32_t top_k;       /* experts per token chosen by the gate (Section 2, k)             */
  int32_t K;           /* resident budget: number of Virtual-Expert slots (#experts_l of  */
                       /* the configuration tuple, Section 3.3); top_k <= K <= E          */
  int32_t dtype;       /* SWAPMOE_F32 or SWAPMOE_BF16: storage type of x, out, weights    */
  int32_t act;         /* SWAPMOE_ACT_RELU: out-proj(relu(in-proj x));                    */
                       /* SWAPMOE_ACT_SWIGLU: out-proj(silu(W1 x) * (W3 x))               */
  int32_t renorm_topk; /* 0: gate value = softmax probability over the allowed experts;   */
                       /* 1: gate value = softmax over the top_k selected logits          */
  int32_t max_tokens;  /* largest n_tokens of any forward; workspace is sized for it      */
  int32_t spare_slots; /* extra arena entries (beyond K) that asynchronous loads may fill */
} swapmoe_config_t;

/* Selectors of swapmoe_debug_copy (intermediates of the LAST forward). */
enum {
  SWAPMOE_TAP_LOGITS = 0, /* fp32 [T, E]                                         */
  SWAPMOE_TAP_UIDX = 1,   /* int32 [T, k]  unmasked top-k experts                */
  SWAPMOE_TAP_UGATE = 2,  /* fp32 [T, k]                                         */
  SWAPMOE_TAP_MIDX = 3,   /* int32 [T, k]  masked (resident-only) top-k experts  */
  SWAPMOE_TAP_MGATE = 4,  /* fp32 [T, k]                                         */
  SWAPMOE_TAP_SLOT = 5,   /* int32 [T, k]                                        */
  SWAPMOE_TAP_COUNT = 6,  /* int32 [K]                                           */
  SWAPMOE_TAP_OFFSET = 7, /* int32 [K+1]                                         */
  SWAPMOE_TAP_PERM = 8,   /* int32 [T*k]   position -> flat pair index t*k+j     */
  SWAPMOE_TAP_INV = 9,    /* int32 [T*k]   flat pair index -> position           */
  SWAPMOE_TAP_XNORM = 10, /* fp32 [T]      L2 norm of every token                */
  /* The next two deliver the T*k occupied rows in POSITION order (row pos belongs to the pair
   * perm[pos]; Section 2, E_i(x) = W_out act(W_in x)).  They exist only when the last forward
   * left them in HBM: H after every forward but the one-launch decode step; Y when GEMM-2 wrote
   * the expert outputs unweighted in one piece, i.e. top_k > 1 on the tensor-core path, or an
   * unsliced contraction on the other paths (top-1 tensor-core layers fold gate * y into `out`).
   * Otherwise the call returns SWAPMOE_ERR_UNSUPPORTED. */
  SWAPMOE_TAP_H = 11,     /* layer dtype [T*k, d_ff]  act(W_in x) of every pair        */
  SWAPMOE_TAP_Y = 12      /* fp32 [T*k, d_model]      W_out h of every pair            */
};

/*
 * Section 3 (online phase): one layer object = one MoE layer served from K
 * resident slots.  Allocates the layer's device workspace (sized for
 * cfg->max_tokens) on the CURRENT CUDA device and zeroes the importance
 * accumulator.  *out is written only on success.  Errors: INVALID_ARG
 * (null, K < top_k, K > E, sizes out of the limits above), UNSUPPORTED, CUDA,
 * NO_MEMORY (the workspace did not fit).
 * Reproducibility: a layer object returns the same bits for the same inputs,
 * tables and weights, call after call and whatever ran before on it (every
 * reduction has a fixed order).  Two layer objects that differ in max_tokens
 * may slice GEMM-2's contraction differently where it is sliced at all (fp32
 * layers, and bf16 layers whose shapes the tcgen05 kernels do not take: the
 * number of partial copies of y follows the workspace size) and then differ
 * in the last bit.
 */
int32_t swapmoe_create(swapmoe_layer_t** out, const swapmoe_config_t* cfg);

/* Frees the workspace.  The caller must have synchronised the streams that used
 * the layer.  NULL is accepted. */
int32_t swapmoe_destroy(swapmoe_layer_t* layer);

/*
 * Section 2 (gate G(x)) and Eq. (1) (||E_i||).  Wr_dev: router matrix [E, d_model]
 * on the device, in the layer's dtype, NOT copied (must outlive the layer's use).
 * enorm_host: E fp32 values ||E_i|| on the host, copied to the device on `stream`
 * before this call returns control (the host array may be reused at once).
 * The norm of an expert's parameters does not depend on the tokens, and
 * non-resident experts are not in HBM, so the caller supplies it.
 */
int32_t swapmoe_set_router(swapmoe_layer_t* layer, const void* Wr_dev, const float* enorm_host,
                           void* stream);

/*
 * Abstract / Section 3: the Virtual-Expert -> actual-expert mapping, and where
 * the resident weights live.
 *   slot_to_expert_host [K]: expert id served by each logical slot (host, copied;
 *       validated: 0 <= id < E, no id twice -> else BAD_SLOT_TABLE).
 *   phys_slot_host [K]: arena entry backing each logical slot, 0 <= p < K +
 *       spare_slots, no entry twice (host, copied); NULL means identity.
 *   arena_in_dev : [K + spare_slots, nin, d_ff, d_model], nin = 1 (ReLU: wi) or
 *       2 (SwiGLU: w1 then w3);  arena_out_dev: [K + spare_slots, d_model, d_ff].
 *       Device memory, layer dtype, caller-owned, not copied.
 * The new tables take effect for forwards enqueued on `stream` after this call;
 * forwards enqueued earlier keep the old tables.  No host synchronisation.
 */
int32_t swapmoe_set_resident(swapmoe_layer_t* layer, const int32_t* slot_to_expert_host,
                             const int32_t* phys_slot_host, const void* arena_in_dev,
                             const void* arena_out_dev, void* stream);

/*
 * The hot path (Sections 2, 3.1; Fig. 4): for every token row of x_dev
 *   logits = x Wr^T;  unmasked top-k gate (feeds Eq. 1);  Masked Gating over the
 *   resident experts;  slot remap;  stable grouping of (token, j) pairs by slot;
 *   grouped expert FFN;  out[t] = sum_j gate[t,j] * E_{slot[t,j]}(x[t]).
 * It also adds this batch's terms of Eq. (1) to the layer's importance
 * accumulator.  out_dev [n_tokens, d_model] is overwritten.  Everything is
 * enqueued on `stream`; the call does not synchronise and does not allocate.
 * n_tokens = 0 is a valid no-op.  Errors: NOT_READY, TOO_MANY_TOKENS,
 * INVALID_ARG, CUDA (launch failure).
 * Launches: four or five kernels; a bf16 layer given at most five (token,
 * expert) pairs (a decode step) runs as a single kernel with the same results
 * and side effects.
 * The router matrix and the arenas must not be written by work enqueued on
 * `stream` immediately before a forward of the same layer (the decode kernel
 * starts fetching the router matrix while its predecessor drains); slot loads
 * go to spare entries on a side stream (swapmoe_load_slot_async).
 */
int32_t swapmoe_forward(swapmoe_layer_t* layer, const void* x_dev, void* out_dev,
                        int32_t n_tokens, void* stream);

/* Same, but the router product is replaced by caller-supplied fp32 logits
 * [n_tokens, E] on the device (test tap: lets routing be compared on identical
 * logits).  x_dev is still needed for ||x|| and the FFN. */
int32_t swapmoe_forward_from_logits(swapmoe_layer_t* layer, const void* x_dev,
                                    const float* logits_dev, void* out_dev, int32_t n_tokens,
                                    void* stream);

/* Measurement form of swapmoe_forward: identical work, but records the
 * SWAPMOE_N_STAGES + 1 caller-owned cudaEvent_t of `events` on `stream` at the
 * stage boundaries (event i before stage i, the last one after the final
 * stage), so a caller can time each kernel of the path with
 * cudaEventElapsedTime.  Stages: 0 router+gate, 1 scan+importance reduce
 * (no launch of its own: the scan and the reductions run inside the permute
 * kernel, so this interval is empty), 2 scan+permute+gather, 3 grouped GEMM-1
 * (+activation), 4 grouped GEMM-2, 5 combine (empty for top-1 bf16 layers,
 * whose GEMM-2 writes the gate-weighted rows itself).  The one-launch decode
 * path records all of its time in stage 0. */
#define SWAPMOE_N_STAGES 6
int32_t swapmoe_forward_timed(swapmoe_layer_t* layer, const void* x_dev, void* out_dev,
                              int32_t n_tokens, void* stream, void* const* events);

/* Measurement aid: launches ONE of the two grouped GEMMs again (`which` = 1: GEMM-1 + activation, 2: GEMM-2) on the
 * state the layer's last swapmoe_forward left behind (its routing, permutation, tile list, gathered rows and hidden
 * activations), on `stream`, so that a caller can time that kernel alone, back to back, with two events around a
 * loop.  `out_dev` must be the `out_dev` of that forward (GEMM-2 of a top-1 layer writes its rows again, with the
 * same values).  Nothing else of the path runs: no router, no permutation, no combine kernel; importance is not
 * touched.  Returns SWAPMOE_ERR_NOT_READY before the first forward and SWAPMOE_ERR_UNSUPPORTED where the last
 * forward had no GEMM launch of its own to repeat (the one-launch decode kernel, the kernels for up to 64 pairs,
 * the warp-level mma fallback).  The paper has no counterpart. */
int32_t swapmoe_debug_rerun_gemm(swapmoe_layer_t* layer, void* out_dev, int32_t which, void* stream);

/* End-to-end form with HOST buffers: copies x_host [n_tokens, d_model] to the
 * device, runs swapmoe_forward, copies the result to out_host, and returns after
 * `stream` has completed.  Pinned host memory makes the copies asynchronous
 * with respect to other streams; pageable memory works but is slower.  It shares
 * the layer's staging buffers with swapmoe_forward_host_async and is ordered
 * behind that call's outstanding work on this layer. */
int32_t swapmoe_forward_host(swapmoe_layer_t* layer, const void* x_host, void* out_host,
                             int32_t n_tokens, void* stream);

/* Pipelined form of swapmoe_forward_host for streams of requests: the copy of x_host (PINNED)
 * into the layer's staging buffer runs on a copy stream owned by the layer, the forward on
 * `stream` behind it, the copy of the result to out_host (PINNED) on a second copy stream; the
 * call returns at once.  x_host must stay untouched, and out_host is defined, only after
 * swapmoe_host_wait(layer) has returned.  Calls on one layer queue up behind each other (one
 * staging buffer each way); calls on different layers overlap their copies with each other's
 * compute.  Same errors as swapmoe_forward_host. */
int32_t swapmoe_forward_host_async(swapmoe_layer_t* layer, const void* x_host, void* out_host,
                                   int32_t n_tokens, void* stream);
/* Blocks until the most recent swapmoe_forward_host_async of this layer has delivered out_host. */
int32_t swapmoe_host_wait(swapmoe_layer_t* layer);

/*
 * Eq. (1): importance(E_i, X) = sum_{x in X_i} ||x|| * |G(x)_i| * ||E_i||, X_i =
 * tokens whose unmasked top-k contains i, accumulated over every forward since
 * the last reset.  Waits for `stream`, copies E fp32 values to imp_host, and if
 * reset != 0 zeroes the accumulator (ordered on `stream`).
 */
int32_t swapmoe_read_importance(swapmoe_layer_t* layer, float* imp_host, int32_t reset,
                                void* stream);

/*
 * Other per-expert scores accumulated next to Eq. (1), read and reset independently:
 *   SWAPMOE_IMP_EQ1        - Eq. (1) over the unmasked routing (what swapmoe_read_importance returns);
 *   SWAPMOE_IMP_COUNT      - number of (token, j) selections per expert under the unmasked routing:
 *                            the token-count score of the "Simple scheduling" ablation (Section 4.4);
 *   SWAPMOE_IMP_EQ1_MASKED - Eq. (1) read literally over the tokens actually passed to each expert,
 *                            i.e. the masked routing (non-resident experts score 0).
 * Same synchronisation and errors as swapmoe_read_importance; unknown kind -> INVALID_ARG.
 */
enum { SWAPMOE_IMP_EQ1 = 0, SWAPMOE_IMP_COUNT = 1, SWAPMOE_IMP_EQ1_MASKED = 2 };
int32_t swapmoe_read_importance_kind(swapmoe_layer_t* layer, int32_t kind, float* imp_host,
                                     int32_t reset, void* stream);

/*
 * Section 2.2 (activation locality: successive tokens use consistent experts), used by the one-launch
 * decode step: while its CTAs route, the kernel pulls the weights of the experts this layer served on
 * its latest steps towards L2 (environment variable SWAPMOE_DECODE_PREFETCH = 1..4 experts; 0, the default, = off),
 * so that a step that asks for the same expert again reads it from cache.  This call reports how often
 * that guess was right: *hits_host of the *touched_host slots served by decode steps since the last reset
 * held a prefetched expert.  Waits for `stream`; reset != 0 zeroes both (ordered on `stream`).
 */
int32_t swapmoe_read_decode_prefetch(swapmoe_layer_t* layer, int64_t* hits_host, int64_t* touched_host,
                                     int32_t reset, void* stream);

/* The same without the wait, for several scores at once: bit k of kinds_mask selects score k
 * (SWAPMOE_IMP_EQ1 = bit 0, SWAPMOE_IMP_COUNT = bit 1, SWAPMOE_IMP_EQ1_MASKED = bit 2).  One small kernel
 * enqueued on `stream` writes score k to scores_host_pinned[k * E .. k * E + E) (PINNED host memory of 3 * E
 * floats, written directly by the device) and, if reset != 0, zeroes the selected accumulators.  The values
 * are there once the caller has synchronised with the stream (an event recorded after this call).  A scheduler
 * can thus read the scores of many layers with one wait, or pick them up a step later without ever stalling
 * the queue of forwards (Section 3.2: updates must not block inference). */
int32_t swapmoe_read_scores_async(swapmoe_layer_t* layer, int32_t kinds_mask, float* scores_host_pinned,
                                  int32_t reset, void* stream);

/*
 * Measurement aid (Section 3.3 profiles an expert's memory traffic; here it is counted): the number
 * of Virtual-Expert slots that received at least one (token, j) pair, summed over every forward
 * since the last reset - i.e. how many experts' weights the layer had to read, the algorithmic
 * weight traffic of the path.  Waits for `stream`; reset != 0 zeroes the counter (ordered on
 * `stream`).
 */
int32_t swapmoe_read_touched_slots(swapmoe_layer_t* layer, int64_t* total_host, int32_t reset,
                                   void* stream);

/* Sections 3.1-3.2: the K most important experts, by descending importance, ties
 * to the lowest index.  Pure host function (E <= 256 floats). */
int32_t swapmoe_topk_importance(const float* imp_host, int32_t E, int32_t K,
                                int32_t* out_idx_host);

/*
 * Section 3.2 (asynchronous expert loading): enqueue on `side_stream` the copy of
 * one expert's matrices from PINNED host memory into arena entry `phys` of the
 * arenas last given to set_resident (in_host_pinned: [nin, d_ff, d_model],
 * out_host_pinned: [d_model, d_ff]), then record `done_event` (may be NULL) on
 * side_stream.  `phys` must not back any logical slot of the table given by the
 * LATEST set_resident (-> BAD_SLOT_TABLE).  Forwards enqueued under an earlier
 * table may still read that entry, so the copy is ordered behind everything
 * enqueued so far on `compute_stream` (the stream the layer's forwards and
 * set_resident calls run on; the call records an event there and makes
 * side_stream wait for it): a forward never reads memory being written.
 * compute_stream must not be capturing.  The caller later makes its compute
 * stream wait on done_event and calls set_resident with a table that uses `phys`.
 */
int32_t swapmoe_load_slot_async(swapmoe_layer_t* layer, int32_t phys, const void* in_host_pinned,
                                const void* out_host_pinned, void* compute_stream,
                                void* side_stream, void* done_event);

/* Copies one intermediate of the last forward to the host after waiting for
 * `stream`.  `bytes` must equal the tap's size for the last n_tokens. */
int32_t swapmoe_debug_copy(swapmoe_layer_t* layer, int32_t which, void* host, size_t bytes,
                           void* stream);

/* Waits for `stream` and returns the device-side status word of the layer:
 * SWAPMOE_OK, or SWAPMOE_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel
 * gave up since the last call.  *detail (may be NULL) receives a code naming
 * the wait.  The word is cleared. */
int32_t swapmoe_device_status(swapmoe_layer_t* layer, int32_t* detail, void* stream);

/* Failure-detection self-test.  Launches one small kernel in which a single thread waits on an
 * mbarrier that nothing will ever complete, through the same bounded wait the tensor-core
 * kernels use but with a limit of limit_ms (1..1000) milliseconds.  The wait must give up: the
 * kernel then returns normally and the layer's status word reads SWAPMOE_ERR_DEVICE_TIMEOUT
 * with detail 99 at the next swapmoe_device_status; the CUDA context stays usable. */
int32_t swapmoe_selftest_bounded_wait(swapmoe_layer_t* layer, int32_t limit_ms, void* stream);

/* Number of kernels of this library launched by the layer so far (host counter). */
int64_t swapmoe_launch_count(const swapmoe_layer_t* layer);

/* Bytes of device workspace the layer allocated at create. */
int64_t swapmoe_workspace_bytes(const swapmoe_layer_t* layer);

/* Selects the grouped-GEMM implementation for later forwards (test / benchmark
 * hook): 0 = automatic, 1 = warp-level mma tiles (the kernels that serve shapes
 * the tcgen05 kernels do not take), 2 = tcgen05 tensor-core tiles (bf16 only;
 * UNSUPPORTED otherwise). */
int32_t swapmoe_set_gemm_path(swapmoe_layer_t* layer, int32_t path);

/*
 * Routing without any allocation.  (The paper has no counterpart of this call: it
 * exists for the way some programs have to use a GPU.)
 *
 * Who needs it: code that runs where cudaMalloc may not be called - a plug-in
 * living inside a host application that owns all device memory and forbids
 * allocations after start-up, a real-time loop that must not take the driver's
 * allocation lock, or a caller that is already inside a region where the CUDA
 * runtime refuses to allocate.  Such callers cannot use swapmoe_create(), which
 * allocates the layer's workspace.  This call runs the router stage alone -
 * logits = x Wr^T, the unmasked and the masked top-k gate, the slot of every
 * routed pair, ||x||, the per-slot counts and their exclusive scan, and this
 * batch's terms of Eq. (1) added into imp_dev - and keeps the few hundred KB of
 * scratch it needs (per-block histograms and partial sums) in a fixed array that
 * is part of the library image.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 *
 * The price of the fixed array: every GPU that loads the library holds it
 * (about 0.35 MB) until the process exits; n_tokens is limited to
 * SWAPMOE_ROUTE_STATIC_MAX_TOKENS (more -> SWAPMOE_ERR_TOO_MANY_TOKENS, E > 256,
 * K > 64, top_k > 4 or d_model not a multiple of 64 -> SWAPMOE_ERR_UNSUPPORTED);
 * and all calls on one GPU share it, so two calls whose kernels may overlap on
 * the device (different streams, or different host threads) race: issue them
 * one after the other on one stream.  The array keeps the previous call's
 * contents; the call itself clears the parts that must start at zero.
 *
 * The first call on each device looks up the array's device address (with that
 * device current); that first call should be made before any stream capture
 * begins.
 *
 * All pointers are device pointers owned by the caller: inputs x_dev
 * [n_tokens, d_model] and Wr_dev [E, d_model] in `dtype` (16-byte aligned),
 * expert_to_slot_dev [E] int32 (-1 = not resident; exactly K entries >= 0),
 * enorm_dev [E] fp32; outputs logits_dev [n_tokens, E] fp32, uidx / midx /
 * slot [n_tokens, top_k] int32, ugate / mgate [n_tokens, top_k] fp32, xnorm_dev
 * [n_tokens] fp32, count_dev [K] and offset_dev [K + 1] int32; imp_dev [E] fp32
 * is accumulated in place (zero it for a fresh score).  Work is enqueued on
 * `stream`; no host synchronisation.  n_tokens = 0 is a no-op.
 */
#define SWAPMOE_ROUTE_STATIC_MAX_TOKENS 8192
int32_t swapmoe_route_static(const void* x_dev, const void* Wr_dev, const int32_t* expert_to_slot_dev,
                             const float* enorm_dev, int32_t n_tokens, int32_t d_model, int32_t E,
                             int32_t top_k, int32_t K, int32_t dtype, int32_t renorm_topk,
                             float* logits_dev, int32_t* uidx_dev, float* ugate_dev, int32_t* midx_dev,
                             float* mgate_dev, int32_t* slot_dev, float* xnorm_dev, int32_t* count_dev,
                             int32_t* offset_dev, float* imp_dev, void* stream);

const char* swapmoe_status_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* SWAPMOE_H_ */
