/*
 * CPU oracle for the cache-conditional MoE decode step ("Mixture of Cache-Conditional Experts").
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA library is checked
 * against.  It shares no code, header, table or constant with the CUDA path and must never be called
 * from the product path; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything here follows the paper's order and notation, one scalar loop per formula:
 *   Eq. 1      y = sum_{i in r[:K]} w_i E_i(x)                      -> orc_ffn_slab / orc_expert_ffn
 *   Eq. 2-3    r = argsort(w), w = softmax(z), z = G(x)             -> orc_router_logits, orc_route_slab
 *   Eq. 4      hit_rate = count(r[:K] ∩ C) / K (cache before token) -> miss counters in orc_route_slab
 *   Sec. 3.1   promote(r_subset; r_all), Eq. 5-6 / Algorithm 1      -> orc_promote, orc_max_rank
 *   Algorithm 2 cumulative-probability threshold                    -> orc_cumsum_threshold
 *   Eq. 7      z' = z + lambda * Delta_avg * m~_t (top-J OR-ed in)  -> orc_route_slab
 *   Eq. 8      Delta_avg = running mean of max(z) - min(z)          -> orc_route_slab
 *   Sec. 4.2   LRU eviction; inside one token the expert with the
 *              higher router weight counts as older                -> orc_route_slab
 *   Sec. 4.8   Belady's farthest-next-use eviction (lossless bound) -> orc_belady_misses
 *
 * Pinned (tests/test_oracle_pins.py): lambda=0 and J=K reduce to plain top-K; C>=E leaves only
 * compulsory misses; the saturated bias equals the list promote operator; the appendix's worked
 * Max-Rank example; LRU against two independent re-implementations; Belady against exhaustive search;
 * weights against a library softmax; the FFN against a float64 library SwiGLU.
 * Parity unpinned: the paper's measured miss rates, lifetimes, perplexities and speed-ups (they need
 * its datasets and checkpoints).
 *
 * Arithmetic: fp32 where the routing decision depends on it (each operation a single IEEE
 * round-to-nearest op: build with -ffp-contract=off), double accumulation for every contraction.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_E 1024

typedef struct {
  int32_t n_layers, n_experts, top_k, top_j, n_shared; /* L, N (=E), K, J, shared experts          */
  int32_t d_model, d_ff, cache_capacity, n_streams;    /* d, I, C, S                               */
  float lambda;                                        /* promotion strength, Eq. 7                */
  int32_t delta_mode;                                  /* 0 running mean (Eq. 8), 1 fixed per layer */
  int32_t renorm;                                      /* 1: weights renormalised over the selected */
  int32_t dtype;                                       /* 0: fp32 everywhere, 1: bf16 hidden+weights */
  int32_t rerank_mode;                                 /* 0 Cache-Prior (Eq. 7), 1 Max-Rank (Alg. 1),
                                                          2 Cumsum-Threshold (Alg. 2)               */
  int32_t max_rank;                                    /* M of Algorithm 1                          */
  float cum_threshold;                                 /* p of Algorithm 2                          */
} orc_config;

void orc_max_rank(const int32_t* r, int n, const uint8_t* in_cache, int M, int J, int32_t* out);

/* ---------------------------------------------------------------------------------------------- */
/* small helpers                                                                                   */

static float bf16_bits_to_float(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Round a double to the nearest value with an 8-bit significand (bfloat16), ties to even. */
static double round_to_bf16(double v) {
  if (v == 0.0 || !isfinite(v)) return v;
  int e;
  double m = frexp(v, &e);              /* v = m * 2^e, 0.5 <= |m| < 1 */
  if (e < -125) return (double)(float)v; /* below bf16's normal range: not reached by the workloads */
  double q = nearbyint(ldexp(m, 8));    /* default rounding mode: ties to even */
  return ldexp(q, e - 8);
}

/* a precedes b in a descending sort with ties broken by the lower expert index */
static int precedes(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

/* first `count` entries of argsort_desc(v), ties -> lower index (Eq. 2) */
static void top_by_value(const float* v, int n, int count, int32_t* out) {
  uint8_t taken[ORC_MAX_E];
  memset(taken, 0, (size_t)n);
  for (int r = 0; r < count; ++r) {
    int best = -1;
    for (int e = 0; e < n; ++e) {
      if (taken[e]) continue;
      if (best < 0 || precedes(v[e], e, v[best], best)) best = e;
    }
    out[r] = best;
    taken[best] = 1;
  }
}

/* Sec. 3.2 (Cumsum-Threshold): the number M of top-ranked experts to consider is the smallest one whose
   router probabilities add up to at least p; all n if they never do.  w_by_rank[i] is the probability of
   the expert of rank i.  mass[i] = probability of the first i ranks, added rank by rank in fp32; M is the
   first i with mass[i] >= p.  *distance (optional) receives how far p lies from the two partial sums on
   either side of the decision, mass[M] - p and p - mass[M-1], whichever is smaller (infinite when M = 0 or
   when p is never reached): a step with a tiny distance could resolve either way in another arithmetic. */
static int ranks_for_mass(const float* w_by_rank, int n, float p, float* distance) {
  float mass[ORC_MAX_E + 1];
  mass[0] = 0.0f;
  for (int i = 0; i < n; ++i) mass[i + 1] = mass[i] + w_by_rank[i];
  int M = n, reached = 0;
  for (int i = n; i >= 0; --i)
    if (mass[i] >= p) M = i, reached = 1;
  if (distance) *distance = (reached && M > 0) ? fminf(mass[M] - p, p - mass[M - 1]) : INFINITY;
  return M;
}

/* ---------------------------------------------------------------------------------------------- */
/* Eq. 3: z = G(x) = W_r x, accumulated in double, rounded once to fp32.                            */
/* x_dtype: 0 = fp32, 1 = bf16 stored as uint16.                                                    */
void orc_router_logits(const float* Wr /*[E,d]*/, const void* x, int x_dtype, int E, int d,
                       float* z /*[E]*/) {
  for (int e = 0; e < E; ++e) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) {
      double xj = x_dtype ? (double)bf16_bits_to_float(((const uint16_t*)x)[j])
                          : (double)((const float*)x)[j];
      acc += (double)Wr[(size_t)e * d + j] * xj;
    }
    z[e] = (float)acc;
  }
}

void orc_router_logits_slab(const orc_config* c, const float* Wr /*[L,E,d]*/,
                            const void* hidden /*[L,S,d]*/, float* z /*[L,S,E]*/, int s0, int s1) {
  const int L = c->n_layers, E = c->n_experts, d = c->d_model, S = c->n_streams;
  const size_t xsz = c->dtype ? 2 : 4;
  for (int l = 0; l < L; ++l)
    for (int s = s0; s < s1; ++s)
      orc_router_logits(Wr + (size_t)l * E * d,
                        (const char*)hidden + ((size_t)l * S + s) * d * xsz, c->dtype, E, d,
                        z + ((size_t)l * S + s) * E);
}

/* ---------------------------------------------------------------------------------------------- */
/* One token of the routing recurrence for every (layer, stream) with s0 <= stream < s1.            */
/*                                                                                                  */
/* State per (layer, stream), all caller-owned flat arrays:                                         */
/*   stamp[E] int64  0 = not in the cache, else the key of the last touch (larger = more recent)    */
/*   ever[E]  uint8  expert has been in the cache at some point (separates compulsory misses)       */
/*   sum_range float, count int64   numerator / denominator of the running Delta_avg (Eq. 8)        */
/*   tok int64       tokens processed so far                                                        */
/*   counters int64[4]  {steps, selections, misses, cold_misses}                                    */
/* Outputs per (layer, stream): sel[K] in rank order of z', w[K] weights from the unmodified z,      */
/* margin = smallest gap that decided an outcome (for near-tie reporting), delta_used.              */
void orc_route_slab(const orc_config* c, const float* z_all /*[L,S,E]*/,
                    const float* fixed_delta /*[L] or NULL*/, int64_t* stamp_all /*[L,S,E]*/,
                    uint8_t* ever_all /*[L,S,E]*/, float* sum_range_all /*[L,S]*/,
                    int64_t* count_all /*[L,S]*/, int64_t* tok_all /*[L,S]*/,
                    int64_t* counters_all /*[L,S,4]*/, int32_t* sel_all /*[L,S,K]*/,
                    float* w_all /*[L,S,K]*/, float* margin_all /*[L,S] or NULL*/,
                    float* delta_all /*[L,S] or NULL*/, int64_t* load_tok_all /*[L,S,E] or NULL*/,
                    int64_t* life_all /*[L,S,3] or NULL: evictions, sum and sum of squares of lifetimes*/,
                    uint32_t* miss_mask_all /*[L,S] or NULL: bit k set iff the k-th selected expert missed*/,
                    int s0, int s1) {
  const int L = c->n_layers, E = c->n_experts, K = c->top_k, J = c->top_j, S = c->n_streams;
  const int C = c->cache_capacity;
  for (int l = 0; l < L; ++l) {
    for (int s = s0; s < s1; ++s) {
      const size_t p = (size_t)l * S + s;
      const float* z = z_all + p * E;
      int64_t* stamp = stamp_all + p * E;
      uint8_t* ever = ever_all + p * E;
      int32_t* sel = sel_all + p * K;
      float* w = w_all + p * K;

      /* Eq. 8: range of the logits of this token, folded into the running mean (inclusive). */
      float zmax = z[0], zmin = z[0];
      for (int e = 1; e < E; ++e) {
        if (z[e] > zmax) zmax = z[e];
        if (z[e] < zmin) zmin = z[e];
      }
      const float range = zmax - zmin;
      float delta;
      if (c->delta_mode == 0) {
        sum_range_all[p] = sum_range_all[p] + range;
        count_all[p] += 1;
        delta = sum_range_all[p] / (float)count_all[p];
      } else {
        delta = fixed_delta[l];
      }

      /* m~_t: cache state after the previous token, OR the top-J experts of the router. */
      int32_t topj[ORC_MAX_E];
      uint8_t mask[ORC_MAX_E];
      top_by_value(z, E, J, topj);
      for (int e = 0; e < E; ++e) mask[e] = stamp[e] != 0;
      for (int j = 0; j < J; ++j) mask[topj[j]] = 1;

      /* Eq. 7: z' = z + lambda * Delta_avg * m~_t. */
      const float bias = c->lambda * delta;
      float zp[ORC_MAX_E];
      for (int e = 0; e < E; ++e) zp[e] = mask[e] ? z[e] + bias : z[e];

      /* r' = argsort(z'); the first K are selected. */
      int32_t rank[ORC_MAX_E];
      const int need = K < E ? K + 1 : K;
      float cum_margin = INFINITY;
      if (c->rerank_mode == 0) {
        top_by_value(zp, E, need, rank);
      } else {
        /* The two baselines rerank the router's own ranking r with the list operator of Sec. 3.1. */
        int32_t r[ORC_MAX_E];
        uint8_t in_cache[ORC_MAX_E];
        top_by_value(z, E, E, r);
        for (int e = 0; e < E; ++e) in_cache[e] = stamp[e] != 0;
        int M = c->max_rank;
        if (c->rerank_mode == 2) {
          /* Algorithm 2 / Sec. 3.2: M from the router probabilities (softmax of z) in rank order. */
          double denom = 0.0;
          float w_by_rank[ORC_MAX_E];
          for (int e = 0; e < E; ++e) denom += exp((double)z[e] - (double)zmax);
          for (int i = 0; i < E; ++i) w_by_rank[i] = (float)(exp((double)z[r[i]] - (double)zmax) / denom);
          M = ranks_for_mass(w_by_rank, E, c->cum_threshold, &cum_margin);
        }
        orc_max_rank(r, E, in_cache, M, J, rank);
      }
      for (int k = 0; k < K; ++k) sel[k] = rank[k];

      /* Expert weights: softmax of the UNMODIFIED logits (Eq. 3), optionally renormalised over
         the selected experts. */
      double denom_all = 0.0, denom_sel = 0.0;
      for (int e = 0; e < E; ++e) denom_all += exp((double)z[e] - (double)zmax);
      for (int k = 0; k < K; ++k) denom_sel += exp((double)z[sel[k]] - (double)zmax);
      for (int k = 0; k < K; ++k)
        w[k] = (float)(exp((double)z[sel[k]] - (double)zmax) / (c->renorm ? denom_sel : denom_all));

      /* Eq. 4 against the cache as it was before this token. */
      int64_t* cnt = counters_all + p * 4;
      int miss = 0, cold = 0;
      uint32_t miss_mask = 0;
      for (int k = 0; k < K; ++k) {
        if (stamp[sel[k]] == 0) ++miss;
        if (stamp[sel[k]] == 0) miss_mask |= 1u << k;
        if (!ever[sel[k]]) ++cold;
      }
      if (miss_mask_all) miss_mask_all[p] = miss_mask;
      cnt[0] += 1;
      cnt[1] += K;
      cnt[2] += miss;
      cnt[3] += cold;

      /* LRU touch.  The K experts of one token are used in parallel; the paper orders them so that
         the one with the higher router weight is evicted first, i.e. is the older one. */
      float zsel[ORC_MAX_E];
      int32_t order[ORC_MAX_E];
      for (int k = 0; k < K; ++k) zsel[k] = z[sel[k]];
      {
        uint8_t taken[ORC_MAX_E];
        memset(taken, 0, (size_t)K);
        for (int r = 0; r < K; ++r) {
          int best = -1;
          for (int k = 0; k < K; ++k) {
            if (taken[k]) continue;
            if (best < 0 || precedes(zsel[k], sel[k], zsel[best], sel[best])) best = k;
          }
          order[r] = best; /* order[0] = highest router weight = oldest inside the token */
          taken[best] = 1;
        }
      }
      const int64_t tok = tok_all[p];
      for (int r = 0; r < K; ++r) {
        const int e = sel[order[r]];
        if (stamp[e] == 0 && load_tok_all) load_tok_all[p * E + e] = tok; /* loaded by this token */
        stamp[e] = (int64_t)E + tok * K + r + 1;
        ever[e] = 1;
      }
      tok_all[p] = tok + 1;

      /* evict least-recently used until the capacity holds */
      for (;;) {
        int resident = 0, victim = -1;
        for (int e = 0; e < E; ++e) {
          if (stamp[e] == 0) continue;
          ++resident;
          if (victim < 0 || stamp[e] < stamp[victim]) victim = e;
        }
        if (resident <= C) break;
        stamp[victim] = 0;
        if (life_all) {
          /* cache lifetime: tokens from the load of an expert to its eviction (Table 2 of the paper) */
          const int64_t life = tok - load_tok_all[p * E + victim];
          life_all[p * 3 + 0] += 1;
          life_all[p * 3 + 1] += life;
          life_all[p * 3 + 2] += life * life;
        }
      }

      if (delta_all) delta_all[p] = delta;
      if (margin_all) {
        /* the smallest gap that decided something: K-th vs (K+1)-th of z', J-th vs (J+1)-th of z,
           and neighbours in the in-token touch order */
        float m = INFINITY;
        if (K < E && c->rerank_mode == 0) m = fminf(m, zp[rank[K - 1]] - zp[rank[K]]);
        if (c->rerank_mode != 0) {
          /* any two neighbours of the router's ranking may swap; the cumulative threshold may fall
             on either side */
          int32_t r[ORC_MAX_E];
          top_by_value(z, E, E, r);
          for (int i = 0; i + 1 < E; ++i) m = fminf(m, z[r[i]] - z[r[i + 1]]);
          m = fminf(m, cum_margin);
        }
        if (J > 0 && J < E) {
          int32_t tj[ORC_MAX_E];
          top_by_value(z, E, J + 1, tj);
          m = fminf(m, z[tj[J - 1]] - z[tj[J]]);
        }
        for (int r = 0; r + 1 < K; ++r) m = fminf(m, zsel[order[r]] - zsel[order[r + 1]]);
        margin_all[p] = m;
      }
    }
  }
}

/* Cache state of one (layer, stream) as the recency-ordered list of resident experts, most recent
   first, padded with -1 to C entries. */
void orc_export_order(const int64_t* stamp /*[E]*/, int E, int C, int32_t* order /*[C]*/) {
  uint8_t taken[ORC_MAX_E];
  memset(taken, 0, (size_t)E);
  for (int r = 0; r < C; ++r) {
    int best = -1;
    for (int e = 0; e < E; ++e) {
      if (taken[e] || stamp[e] == 0) continue;
      if (best < 0 || stamp[e] > stamp[best]) best = e;
    }
    order[r] = best;
    if (best >= 0) taken[best] = 1;
  }
}

/* Initial cache content (empty, or a given set): `order` lists resident experts most recent first,
   -1 padded.  These entries are older than anything touched later. */
void orc_import_order(const int32_t* order /*[C]*/, int E, int C, int64_t* stamp /*[E]*/,
                      uint8_t* ever /*[E]*/) {
  for (int e = 0; e < E; ++e) stamp[e] = 0;
  for (int r = 0; r < C; ++r) {
    if (order[r] < 0) continue;
    stamp[order[r]] = C - r; /* 1..C, all below E + 1 */
    ever[order[r]] = 1;
  }
}

/* ---------------------------------------------------------------------------------------------- */
/* Eq. 1 expert: E_i(x) = W_d ( silu(W_g x) ⊙ (W_u x) ), SwiGLU.  dtype 1: x and all W are bf16      */
/* (uint16 storage) and the intermediate h is rounded to bf16 before the down projection, the       */
/* rounding point of a bf16 tensor-core pipeline; dtype 0: fp32 inputs, no rounding.                */
static double load_elem(const void* base, size_t i, int dtype) {
  return dtype ? (double)bf16_bits_to_float(((const uint16_t*)base)[i])
               : (double)((const float*)base)[i];
}

void orc_expert_ffn(const void* x /*[d]*/, const void* Wg /*[I,d]*/, const void* Wu /*[I,d]*/,
                    const void* Wd /*[d,I]*/, int d, int I, int dtype, double* o /*[d]*/) {
  double* h = (double*)malloc(sizeof(double) * (size_t)I);
  for (int i = 0; i < I; ++i) {
    double g = 0.0, u = 0.0;
    for (int j = 0; j < d; ++j) {
      const double xj = load_elem(x, (size_t)j, dtype);
      g += load_elem(Wg, (size_t)i * d + j, dtype) * xj;
      u += load_elem(Wu, (size_t)i * d + j, dtype) * xj;
    }
    const double silu = g / (1.0 + exp(-g));
    h[i] = dtype ? round_to_bf16(silu * u) : silu * u;
  }
  for (int j = 0; j < d; ++j) {
    double acc = 0.0;
    for (int i = 0; i < I; ++i) acc += load_elem(Wd, (size_t)j * I + i, dtype) * h[i];
    o[j] = acc;
  }
  free(h);
}

/* Eq. 1 for every (layer, stream) with s0 <= stream < s1: routed experts weighted by w in selection
   order, then the always-on shared experts with weight 1. */
void orc_ffn_slab(const orc_config* c, const void* hidden /*[L,S,d]*/,
                  const int32_t* sel /*[L,S,K]*/, const float* w /*[L,S,K]*/,
                  const void* Wg /*[L,E,I,d]*/, const void* Wu /*[L,E,I,d]*/,
                  const void* Wd /*[L,E,d,I]*/, const void* shWg /*[L,n_sh,I,d]*/,
                  const void* shWu, const void* shWd /*[L,n_sh,d,I]*/, float* y /*[L,S,d]*/, int s0,
                  int s1) {
  const int L = c->n_layers, E = c->n_experts, K = c->top_k, S = c->n_streams;
  const int d = c->d_model, I = c->d_ff, nsh = c->n_shared;
  const size_t esz = c->dtype ? 2 : 4;
  const size_t wsz = (size_t)I * d * esz;
  double* o = (double*)malloc(sizeof(double) * (size_t)d);
  double* acc = (double*)malloc(sizeof(double) * (size_t)d);
  for (int l = 0; l < L; ++l) {
    for (int s = s0; s < s1; ++s) {
      const size_t p = (size_t)l * S + s;
      const char* x = (const char*)hidden + p * d * esz;
      for (int j = 0; j < d; ++j) acc[j] = 0.0;
      for (int k = 0; k < K; ++k) {
        const size_t ei = (size_t)l * E + sel[p * K + k];
        orc_expert_ffn(x, (const char*)Wg + ei * wsz, (const char*)Wu + ei * wsz,
                       (const char*)Wd + ei * wsz, d, I, c->dtype, o);
        for (int j = 0; j < d; ++j) acc[j] += (double)w[p * K + k] * o[j];
      }
      for (int q = 0; q < nsh; ++q) {
        const size_t ei = (size_t)l * nsh + q;
        orc_expert_ffn(x, (const char*)shWg + ei * wsz, (const char*)shWu + ei * wsz,
                       (const char*)shWd + ei * wsz, d, I, c->dtype, o);
        for (int j = 0; j < d; ++j) acc[j] += o[j];
      }
      for (int j = 0; j < d; ++j) y[p * d + j] = (float)acc[j];
    }
  }
  free(o);
  free(acc);
}

/* ---------------------------------------------------------------------------------------------- */
/* Sec. 3.1 list operator: promote(subset; all) = subset ⊕ (all \ subset), both orders preserved.   */
void orc_promote(const int32_t* subset, int n_subset, const int32_t* all, int n_all,
                 int32_t* out /*[n_all]*/) {
  int n = 0;
  for (int i = 0; i < n_subset; ++i) out[n++] = subset[i];
  for (int i = 0; i < n_all; ++i) {
    int in_subset = 0;
    for (int j = 0; j < n_subset; ++j)
      if (subset[j] == all[i]) in_subset = 1;
    if (!in_subset) out[n++] = all[i];
  }
}

/* Algorithm 1 (Max-Rank): promote the cached experts among the first M ranks, then the first J
   ranks of the original ranking.  in_cache[e] != 0 marks the cache set C. */
void orc_max_rank(const int32_t* r, int n, const uint8_t* in_cache, int M, int J,
                  int32_t* out /*[n]*/) {
  int32_t subset[ORC_MAX_E], tmp[ORC_MAX_E];
  int ns = 0;
  for (int i = 0; i < M && i < n; ++i)
    if (in_cache[r[i]]) subset[ns++] = r[i];
  orc_promote(subset, ns, r, n, tmp);
  orc_promote(r, J, tmp, n, out);
}

/* Algorithm 2 / Sec. 3.2 (Cumsum-Threshold): Max-Rank with M = the smallest number of top ranks whose
   router probabilities sum to at least p.  w[e] are the softmax weights; returns the M it used. */
int orc_cumsum_threshold(const int32_t* r, int n, const float* w, const uint8_t* in_cache, float p,
                         int J, int32_t* out /*[n]*/) {
  float w_by_rank[ORC_MAX_E];
  for (int i = 0; i < n; ++i) w_by_rank[i] = w[r[i]];
  const int M = ranks_for_mass(w_by_rank, n, p, NULL);
  orc_max_rank(r, n, in_cache, M, J, out);
  return M;
}

/* ---------------------------------------------------------------------------------------------- */
/* Belady's rule for a trace of K-expert requests (one set per token): on a miss evict, among the   */
/* cached experts not requested by the current token, the one whose next use lies farthest ahead.   */
/* Requires C >= K.  Returns the number of misses; the cache starts empty.                          */
int64_t orc_belady_misses(const int32_t* trace /*[T,K]*/, int T, int K, int E, int C) {
  uint8_t in_cache[ORC_MAX_E];
  memset(in_cache, 0, (size_t)E);
  int64_t misses = 0;
  for (int t = 0; t < T; ++t) {
    const int32_t* req = trace + (size_t)t * K;
    for (int k = 0; k < K; ++k) {
      if (in_cache[req[k]]) continue;
      ++misses;
      in_cache[req[k]] = 1;
    }
    for (;;) {
      int resident = 0;
      for (int e = 0; e < E; ++e) resident += in_cache[e];
      if (resident <= C) break;
      int victim = -1;
      int64_t victim_next = -1;
      for (int e = 0; e < E; ++e) {
        if (!in_cache[e]) continue;
        int pinned = 0;
        for (int k = 0; k < K; ++k)
          if (req[k] == e) pinned = 1;
        if (pinned) continue;
        int64_t next = (int64_t)T + 1; /* never used again */
        for (int u = t + 1; u < T && next > T; ++u)
          for (int k = 0; k < K; ++k)
            if (trace[(size_t)u * K + k] == e) next = u;
        if (next > victim_next) {
          victim_next = next;
          victim = e;
        }
      }
      in_cache[victim] = 0;
    }
  }
  return misses;
}

/* Plain LRU on the same kind of trace, touch order inside a token as given (first = oldest).
   Used to compare eviction policies on a fixed, lossless trace. */
int64_t orc_lru_misses(const int32_t* trace /*[T,K]*/, int T, int K, int E, int C) {
  int64_t stamp[ORC_MAX_E];
  memset(stamp, 0, sizeof(int64_t) * (size_t)E);
  int64_t misses = 0;
  for (int t = 0; t < T; ++t) {
    const int32_t* req = trace + (size_t)t * K;
    for (int k = 0; k < K; ++k)
      if (stamp[req[k]] == 0) ++misses;
    for (int k = 0; k < K; ++k) stamp[req[k]] = (int64_t)t * K + k + 1;
    for (;;) {
      int resident = 0, victim = -1;
      for (int e = 0; e < E; ++e) {
        if (stamp[e] == 0) continue;
        ++resident;
        if (victim < 0 || stamp[e] < stamp[victim]) victim = e;
      }
      if (resident <= C) break;
      stamp[victim] = 0;
    }
  }
  return misses;
}
