/*
 * CPU oracle for the Virtual-Expert MoE-layer forward of SwapMoE (arXiv 2308.15030).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the layer computes.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference leg may call it; the product (the CUDA
 * library) shares no code with it and never routes through it.
 *
 * Every function takes host pointers.  Stored inputs (tokens, router, expert
 * matrices) arrive as float32 holding values exactly representable in the
 * layer's storage type and are widened to double before any arithmetic.  There
 * is no blocking, fusion or reordering: each step is the definition, written as
 * loops, in the order the paper's Sections 2 and 3.1 give them.
 *
 * Pins (tests/test_oracle_pins.py): brute-force dense-then-mask evaluation on
 * tiny inputs, the K = E reduction to the unrestricted layer (Section 2,
 * y = G(x)_i E_i(x)), the E = K = 1 reduction to a dense MLP, routing
 * invariants, gate normalisation, token-order invariance and closed forms of
 * Eq. (1).  The paper prints no worked numeric example of one layer, so parity
 * with the paper's own end-to-end figures is "parity unpinned"; what is pinned
 * is the method as read from Sections 2, 3.1 and the Masked-Gating caption of
 * Figure 4.
 *
 * Readings taken where the paper is silent:
 *   - Masked Gating (Fig. 4): non-resident experts get logit -inf before the
 *     softmax, so the gate is a softmax over the resident set.
 *   - Eq. (1) uses the UNMASKED routing for the token set X_i (otherwise an
 *     absent expert could never gain importance and Section 3.2 could not swap
 *     it in); ||G(x)_i|| is |gate value|, ||x|| the token's L2 norm, ||E_i|| a
 *     per-expert scalar supplied by the caller.
 *   - ties in any top-k go to the lowest index; the k selections are ordered by
 *     descending logit; no capacity limit, no biases, no residual.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_ACT_RELU 0
#define ORACLE_ACT_SWIGLU 1

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Section 2: the router's pre-softmax scores, logits[t,e] = sum_c x[t,c] * Wr[e,c]. */
void oracle_logits(const float* x, const float* Wr, int T, int d, int E, double* logits) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int e = 0; e < E; ++e) {
      double acc = 0.0;
      for (int c = 0; c < d; ++c) acc += (double)x[(size_t)t * d + c] * (double)Wr[(size_t)e * d + c];
      logits[(size_t)t * E + e] = acc;
    }
  }
}

/*
 * Section 2 (top-k gate G(x)) and Figure 4 (Masked Gating).
 * allowed == NULL: the off-the-shelf gate over all E experts.
 * allowed[e] != 0 marks the resident (Virtual) experts; the others are treated
 * as logit = -inf.  Selection: k largest allowed logits, ties to the lowest
 * index, j = 0 the largest.  Gate value: renorm == 0 -> softmax probability
 * over the allowed set; renorm != 0 -> softmax over the k selected logits.
 * Returns -1 if fewer than k experts are allowed.
 */
int oracle_gate(const double* logits, int T, int E, int k, int renorm,
                const int32_t* allowed, int32_t* idx, double* gate) {
  int n_allowed = 0;
  for (int e = 0; e < E; ++e) n_allowed += (allowed == NULL || allowed[e]) ? 1 : 0;
  if (n_allowed < k || k < 1) return -1;
  for (int t = 0; t < T; ++t) {
    const double* l = logits + (size_t)t * E;
    for (int j = 0; j < k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        if (allowed != NULL && !allowed[e]) continue;
        int taken = 0;
        for (int q = 0; q < j; ++q) taken |= (idx[(size_t)t * k + q] == e);
        if (taken) continue;
        if (best < 0 || l[e] > l[best]) best = e; /* strict '>' keeps the lowest index on ties */
      }
      idx[(size_t)t * k + j] = best;
    }
    const double m = l[idx[(size_t)t * k]]; /* largest allowed logit */
    double den = 0.0;
    if (renorm) {
      for (int j = 0; j < k; ++j) den += exp(l[idx[(size_t)t * k + j]] - m);
    } else {
      for (int e = 0; e < E; ++e)
        if (allowed == NULL || allowed[e]) den += exp(l[e] - m);
    }
    for (int j = 0; j < k; ++j) gate[(size_t)t * k + j] = exp(l[idx[(size_t)t * k + j]] - m) / den;
  }
  return 0;
}

/* Abstract / Section 1: the Virtual-Expert -> actual-expert mapping, inverted.
 * expert_to_slot[e] = s if slot_to_expert[s] == e, else -1. Returns -1 on a bad table. */
int oracle_invert_slot_table(const int32_t* slot_to_expert, int K, int E, int32_t* expert_to_slot) {
  for (int e = 0; e < E; ++e) expert_to_slot[e] = -1;
  for (int s = 0; s < K; ++s) {
    int e = slot_to_expert[s];
    if (e < 0 || e >= E || expert_to_slot[e] != -1) return -1;
    expert_to_slot[e] = s;
  }
  return 0;
}

/* slot[p] = expert_to_slot[midx[p]]; returns -1 if a masked choice is not resident. */
int oracle_remap(const int32_t* midx, int n, const int32_t* expert_to_slot, int32_t* slot) {
  for (int p = 0; p < n; ++p) {
    slot[p] = expert_to_slot[midx[p]];
    if (slot[p] < 0) return -1;
  }
  return 0;
}

/*
 * Grouping of the (token, j) pairs by slot.  Section 2 only says each token may
 * choose a different expert; the order inside a slot is fixed here as ascending
 * flat index p = t*k + j (a stable counting sort), which makes perm unique.
 * count[K], offset[K+1], perm[n] (position -> flat index), inv[n] (flat -> position).
 */
void oracle_permute(const int32_t* slot, int n, int K, int32_t* count, int32_t* offset,
                    int32_t* perm, int32_t* inv) {
  for (int s = 0; s < K; ++s) count[s] = 0;
  for (int p = 0; p < n; ++p) count[slot[p]] += 1;
  offset[0] = 0;
  for (int s = 0; s < K; ++s) offset[s + 1] = offset[s] + count[s];
  int32_t* cursor = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K > 0 ? K : 1));
  for (int s = 0; s < K; ++s) cursor[s] = offset[s];
  for (int p = 0; p < n; ++p) {
    int pos = cursor[slot[p]]++;
    perm[pos] = p;
    inv[p] = pos;
  }
  free(cursor);
}

/*
 * Section 2, E_i(x): one expert FFN applied to one token, no biases.
 *   ReLU   : y = W_out * max(0, W_in * x)
 *   SwiGLU : y = W_out * ( silu(W_1 * x) .* (W_3 * x) ),  silu(a) = a / (1 + exp(-a))
 * w_in is [nin, f, d] (nin = 1 or 2), w_out is [d, f]; contraction index innermost.
 */
static void expert_ffn(const float* xt, const float* w_in, const float* w_out, int d, int f,
                       int act, double* h, double* y) {
  const float* w1 = w_in;
  const float* w3 = w_in + (size_t)f * d;
  for (int r = 0; r < f; ++r) {
    double a = 0.0;
    for (int c = 0; c < d; ++c) a += (double)w1[(size_t)r * d + c] * (double)xt[c];
    if (act == ORACLE_ACT_SWIGLU) {
      double b = 0.0;
      for (int c = 0; c < d; ++c) b += (double)w3[(size_t)r * d + c] * (double)xt[c];
      h[r] = (a / (1.0 + exp(-a))) * b;
    } else {
      h[r] = a > 0.0 ? a : 0.0;
    }
  }
  for (int c = 0; c < d; ++c) {
    double acc = 0.0;
    for (int r = 0; r < f; ++r) acc += (double)w_out[(size_t)c * f + r] * h[r];
    y[c] = acc;
  }
}

/*
 * y[p,:] = E_{slot[p]}(x[p div k,:]) for every pair p, read straight from the
 * flat (token, j) order: the permutation plays no part in the values.
 * arena_in [P, nin, f, d], arena_out [P, d, f]; phys_slot[s] = arena entry of slot s.
 * token_subset == NULL evaluates all T tokens; otherwise only the n_subset listed
 * tokens are evaluated (rows of other tokens are left untouched).
 */
void oracle_expert_outputs(const float* x, int T, int d, int f, int k, int act,
                           const int32_t* slot, const int32_t* phys_slot,
                           const float* arena_in, const float* arena_out,
                           const int32_t* token_subset, int n_subset, double* y) {
  const int nin = (act == ORACLE_ACT_SWIGLU) ? 2 : 1;
  const int n = token_subset ? n_subset : T;
#pragma omp parallel
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)f);
#pragma omp for schedule(dynamic, 1)
    for (int i = 0; i < n; ++i) {
      const int t = token_subset ? token_subset[i] : i;
      for (int j = 0; j < k; ++j) {
        const size_t p = (size_t)t * k + j;
        const size_t ph = (size_t)phys_slot[slot[p]];
        expert_ffn(x + (size_t)t * d, arena_in + ph * nin * f * d, arena_out + ph * d * f, d, f,
                   act, h, y + p * d);
      }
    }
    free(h);
  }
}

/*
 * Section 2, the inner half of E_i(x) on its own: h[p,:] = act(W_in[slot[p]] * x[p div k,:])
 * for every pair p in flat (token, j) order, so that the first grouped product of an
 * implementation can be compared by itself.  Same definitions as expert_ffn:
 * ReLU max(0, W_in x); SwiGLU silu(W_1 x) .* (W_3 x).  token_subset as above.
 */
void oracle_expert_hidden(const float* x, int T, int d, int f, int k, int act,
                          const int32_t* slot, const int32_t* phys_slot, const float* arena_in,
                          const int32_t* token_subset, int n_subset, double* h) {
  const int nin = (act == ORACLE_ACT_SWIGLU) ? 2 : 1;
  const int n = token_subset ? n_subset : T;
#pragma omp parallel for schedule(dynamic, 1)
  for (int i = 0; i < n; ++i) {
    const int t = token_subset ? token_subset[i] : i;
    const float* xt = x + (size_t)t * d;
    for (int j = 0; j < k; ++j) {
      const size_t p = (size_t)t * k + j;
      const float* w1 = arena_in + (size_t)phys_slot[slot[p]] * nin * f * d;
      const float* w3 = w1 + (size_t)f * d;
      for (int r = 0; r < f; ++r) {
        double a = 0.0;
        for (int c = 0; c < d; ++c) a += (double)w1[(size_t)r * d + c] * (double)xt[c];
        if (act == ORACLE_ACT_SWIGLU) {
          double b = 0.0;
          for (int c = 0; c < d; ++c) b += (double)w3[(size_t)r * d + c] * (double)xt[c];
          h[p * f + r] = (a / (1.0 + exp(-a))) * b;
        } else {
          h[p * f + r] = a > 0.0 ? a : 0.0;
        }
      }
    }
  }
}

/* Section 2: out[t,:] = sum_j G(x_t)_j * E_j(x_t)  (for k = 1: y = G(x)_i E_i(x)). */
void oracle_combine(const double* y, const double* mgate, int T, int d, int k,
                    const int32_t* token_subset, int n_subset, double* out) {
  const int n = token_subset ? n_subset : T;
  for (int i = 0; i < n; ++i) {
    const int t = token_subset ? token_subset[i] : i;
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int j = 0; j < k; ++j) acc += mgate[(size_t)t * k + j] * y[((size_t)t * k + j) * d + c];
      out[(size_t)t * d + c] = acc;
    }
  }
}

/*
 * Eq. (1): importance(E_i, X) = sum over x in X_i of ||x|| * |G(x)_i| * ||E_i||,
 * X_i = tokens whose (unmasked) top-k contains i.  imp[E] is accumulated in place.
 */
void oracle_importance(const float* x, int T, int d, int k, const int32_t* uidx,
                       const double* ugate, const float* enorm, double* imp) {
  for (int t = 0; t < T; ++t) {
    double ss = 0.0;
    for (int c = 0; c < d; ++c) ss += (double)x[(size_t)t * d + c] * (double)x[(size_t)t * d + c];
    const double xn = sqrt(ss);
    for (int j = 0; j < k; ++j) {
      const int e = uidx[(size_t)t * k + j];
      imp[e] += xn * fabs(ugate[(size_t)t * k + j]) * (double)enorm[e];
    }
  }
}

/* "Simple scheduling" ablation of Section 4.4: importance = number of tokens routed. */
void oracle_importance_count(int T, int k, const int32_t* uidx, double* imp) {
  for (int p = 0; p < T * k; ++p) imp[uidx[p]] += 1.0;
}

/* Section 3.1/3.2: the K most important experts, ties to the lowest index,
 * listed by descending importance. */
void oracle_topk_importance(const double* imp, int E, int K, int32_t* out_idx) {
  for (int j = 0; j < K; ++j) {
    int best = -1;
    for (int e = 0; e < E; ++e) {
      int taken = 0;
      for (int q = 0; q < j; ++q) taken |= (out_idx[q] == e);
      if (taken) continue;
      if (best < 0 || imp[e] > imp[best]) best = e;
    }
    out_idx[j] = best;
  }
}

/*
 * The whole layer, steps in the paper's order.  ext_logits (float32, may be NULL)
 * replaces step 1 so routing can be compared on identical logits.
 * Outputs (any may be NULL except out): logits[T,E], uidx/ugate[T,k], midx/mgate[T,k],
 * slot[T,k], count[K], offset[K+1], perm[T*k], inv[T*k], y[T*k,d], out[T,d];
 * imp[E] is accumulated in place.  Returns 0, or -1 on an invalid slot table / K < k.
 */
int oracle_forward(const float* x, const float* Wr, const float* ext_logits, const float* enorm,
                   const int32_t* slot_to_expert, const int32_t* phys_slot,
                   const float* arena_in, const float* arena_out,
                   int T, int d, int f, int E, int k, int K, int act, int renorm,
                   const int32_t* token_subset, int n_subset,
                   double* logits_out, int32_t* uidx_out, double* ugate_out,
                   int32_t* midx_out, double* mgate_out, int32_t* slot_out,
                   int32_t* count_out, int32_t* offset_out, int32_t* perm_out, int32_t* inv_out,
                   double* y_out, double* out, double* imp) {
  const size_t n = (size_t)T * k;
  int rc = 0;
  double* logits = (double*)malloc(sizeof(double) * ((size_t)T * E + 1));
  int32_t* uidx = (int32_t*)malloc(sizeof(int32_t) * (n + 1));
  int32_t* midx = (int32_t*)malloc(sizeof(int32_t) * (n + 1));
  int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * (n + 1));
  int32_t* perm = (int32_t*)malloc(sizeof(int32_t) * (n + 1));
  int32_t* inv = (int32_t*)malloc(sizeof(int32_t) * (n + 1));
  int32_t* count = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K + 1));
  int32_t* offset = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K + 2));
  int32_t* e2s = (int32_t*)malloc(sizeof(int32_t) * (size_t)(E + 1));
  int32_t* allowed = (int32_t*)malloc(sizeof(int32_t) * (size_t)(E + 1));
  double* ugate = (double*)malloc(sizeof(double) * (n + 1));
  double* mgate = (double*)malloc(sizeof(double) * (n + 1));
  double* y = y_out ? y_out : (double*)malloc(sizeof(double) * (n * d + 1));

  /* 1. router scores */
  if (ext_logits) {
    for (size_t i = 0; i < (size_t)T * E; ++i) logits[i] = (double)ext_logits[i];
  } else {
    oracle_logits(x, Wr, T, d, E, logits);
  }
  /* 2. off-the-shelf gate (feeds Eq. 1) */
  if (oracle_gate(logits, T, E, k, renorm, NULL, uidx, ugate) != 0) rc = -1;
  /* 3. Masked Gating over the resident set */
  if (rc == 0 && oracle_invert_slot_table(slot_to_expert, K, E, e2s) != 0) rc = -1;
  if (rc == 0) {
    for (int e = 0; e < E; ++e) allowed[e] = (e2s[e] >= 0);
    if (oracle_gate(logits, T, E, k, renorm, allowed, midx, mgate) != 0) rc = -1;
  }
  /* 4. Virtual-Expert slot of every routed pair */
  if (rc == 0 && oracle_remap(midx, (int)n, e2s, slot) != 0) rc = -1;
  if (rc == 0) {
    /* 5. grouping by slot */
    oracle_permute(slot, (int)n, K, count, offset, perm, inv);
    /* 6. expert FFNs, 7. gate-weighted combine */
    oracle_expert_outputs(x, T, d, f, k, act, slot, phys_slot, arena_in, arena_out,
                          token_subset, n_subset, y);
    oracle_combine(y, mgate, T, d, k, token_subset, n_subset, out);
    /* 8. Eq. (1) */
    if (imp) oracle_importance(x, T, d, k, uidx, ugate, enorm, imp);

    if (logits_out) memcpy(logits_out, logits, sizeof(double) * (size_t)T * E);
    if (uidx_out) memcpy(uidx_out, uidx, sizeof(int32_t) * n);
    if (ugate_out) memcpy(ugate_out, ugate, sizeof(double) * n);
    if (midx_out) memcpy(midx_out, midx, sizeof(int32_t) * n);
    if (mgate_out) memcpy(mgate_out, mgate, sizeof(double) * n);
    if (slot_out) memcpy(slot_out, slot, sizeof(int32_t) * n);
    if (count_out) memcpy(count_out, count, sizeof(int32_t) * (size_t)K);
    if (offset_out) memcpy(offset_out, offset, sizeof(int32_t) * (size_t)(K + 1));
    if (perm_out) memcpy(perm_out, perm, sizeof(int32_t) * n);
    if (inv_out) memcpy(inv_out, inv, sizeof(int32_t) * n);
  }
  free(logits); free(uidx); free(midx); free(slot); free(perm); free(inv); free(count);
  free(offset); free(e2s); free(allowed); free(ugate); free(mgate);
  if (!y_out) free(y);
  return rc;
}
