/*
 * MoIN serving hot path - CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, double-precision statement of what the GPU library computes, written
 * from the paper's definitions so that it can be checked against them by eye:
 *
 *   - the query router: nearest topic embedding of a query embedding (Sec. 3.3), with the
 *     cosine similarity as the metric;
 *   - the LoRA linear layer y = W x + W_b (W_a x) (Sec. 3.2), with the expert chosen per
 *     token (one expert per request, Sec. 3.3), an optional scale s on the low-rank term
 *     and "no adapter => base model only" (Sec. 4, downstream-task paragraph);
 *   - a Llama-architecture decoder forward (Sec. 4 names the base model) in which every one
 *     of the seven per-block projections is that layer;
 *   - the update step of the K-means clustering of document embeddings whose centroids are
 *     the topic embeddings the router searches (Sec. 3.1, second approach; Sec. 4).
 *
 * No blocking, no fusion, no reordering: every sum runs over its index in increasing
 * order.  Parallelism (OpenMP) is only over independent units: queries, tokens, requests.
 * Nothing here shares code, headers, tables or helpers with the CUDA library, and nothing
 * in the CUDA library may call into this file.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 * Pins (tests that tie this file to something other than itself) are in
 * tests/test_oracle_*.py.  Every function has one: the decoder's exact variant is held
 * against the `transformers` Llama implementation in float64 (base model, and each routed
 * request with its adapter merged into the weights), and its storage-rounded variant against
 * a numpy restatement of one block that rounds at exactly the listed points.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F64 0
#define ORACLE_BF16 1

/* Element i of an array stored either as double or as bf16 bit patterns (exact widening). */
static inline double ld(const void* p, int dtype, size_t i) {
  if (dtype == ORACLE_F64) return ((const double*)p)[i];
  uint32_t u = ((uint32_t)((const uint16_t*)p)[i]) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* Round a double to the nearest bf16 value (ties to even), returned as a double.
 * Used only by the decoder's "storage-rounded" variant, at the points where the GPU
 * library keeps a tensor in bf16. */
static double round_bf16(double v) {
  if (isnan(v) || isinf(v) || v == 0.0) return v;
  int ex;
  double m = frexp(v, &ex);           /* v = m * 2^ex, 0.5 <= |m| < 1 */
  if (ex < -125) {                    /* bf16 subnormal range: quantum 2^-133 */
    double q = ldexp(1.0, -133);
    return nearbyint(v / q) * q;
  }
  double scaled = ldexp(m, 8);        /* 8 significant bits: 128 <= |scaled| < 256 */
  double r = nearbyint(scaled);       /* default rounding mode: ties to even */
  double out = ldexp(r, ex - 8);
  if (fabs(out) > 3.3895313892515355e38) out = copysign(INFINITY, v);
  return out;
}

int moin_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

double moin_oracle_round_bf16(double v) { return round_bf16(v); }

/* ------------------------------------------------------------------------------------
 * Router (Sec. 3.3: nearest-neighbour search of the query embedding over the topic
 * embeddings; metric = cosine similarity).
 *
 *   sim[i][k] = <q_i, c_k> / (|q_i| |c_k|)
 *   id[i]     = smallest k attaining max_k sim[i][k]
 *   margin[i] = best - second best (over k != id[i]); +inf when K == 1
 *
 * A zero-norm centroid has similarity -inf, and -inf never wins.  A NaN similarity never
 * wins.  If nothing wins (a zero-norm query, whose similarities are all NaN or -inf; or a
 * table of zero-norm centroids) the id is 0.
 * With centroid_to_expert != NULL, expert[i] = centroid_to_expert[id[i]].
 * ------------------------------------------------------------------------------------ */
int moin_oracle_route(const void* q, const void* c, int dtype, int64_t Q, int64_t K, int64_t D,
                      const int32_t* centroid_to_expert, int32_t* out_centroid,
                      int32_t* out_expert, double* out_best, double* out_margin) {
  if (Q < 0 || K <= 0 || D <= 0) return -1;
  double* cnorm = (double*)malloc(sizeof(double) * (size_t)K);
  if (!cnorm) return -2;
  for (int64_t k = 0; k < K; ++k) {
    double s = 0.0;
    for (int64_t d = 0; d < D; ++d) {
      double v = ld(c, dtype, (size_t)(k * D + d));
      s += v * v;
    }
    cnorm[k] = sqrt(s);
  }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < Q; ++i) {
    double qs = 0.0;
    for (int64_t d = 0; d < D; ++d) {
      double v = ld(q, dtype, (size_t)(i * D + d));
      qs += v * v;
    }
    double qn = sqrt(qs);
    double best = -INFINITY, second = -INFINITY;
    int64_t id = 0;
    int won = 0;
    for (int64_t k = 0; k < K; ++k) {
      double dot = 0.0;
      for (int64_t d = 0; d < D; ++d)
        dot += ld(q, dtype, (size_t)(i * D + d)) * ld(c, dtype, (size_t)(k * D + d));
      double sim = (cnorm[k] == 0.0) ? -INFINITY : dot / (qn * cnorm[k]);
      if (isnan(sim)) continue;
      if (sim > best) {          /* strict: lowest index on ties; -inf never wins */
        second = best;
        best = sim;
        id = k;
        won = 1;
      } else if (sim > second) {
        second = sim;
      }
    }
    if (out_centroid) out_centroid[i] = (int32_t)id;
    if (out_expert) out_expert[i] = centroid_to_expert ? centroid_to_expert[id] : (int32_t)id;
    if (out_best) out_best[i] = won ? best : NAN;
    if (out_margin) out_margin[i] = (K == 1 || !won) ? INFINITY : best - second;
  }
  free(cnorm);
  return 0;
}

/* ------------------------------------------------------------------------------------
 * Routed LoRA linear layer (Sec. 3.2, y = W x + W_b (W_a x), W in R^{k x d},
 * W_a in R^{r x d}, W_b in R^{k x r}; expert per request, Sec. 3.3).
 *
 * Storage: x[T][d_in], W[d_out][d_in], A[n_slots][r][d_in] (= W_a of each stored adapter),
 * B[n_slots][d_out][r] (= W_b), token_expert[T], slot_of_expert[E].
 * For token t with expert e = token_expert[t]:
 *   slot = slot_of_expert[e] if 0 <= e < E else -1
 *   y[t][j] = sum_i W[j][i] x[t][i]  (+ s * sum_p B[slot][j][p] * (sum_i A[slot][p][i] x[t][i])
 *                                      if slot >= 0)
 * y is left in double.  One token per loop iteration; tokens are independent.
 * ------------------------------------------------------------------------------------ */
/* Optional function between the two low-rank matrices (the paper's formula has none; Sec. 5 lists "an
 * activation between the two LoRA matrices" as a variant): y = W x + s W_b act(W_a x). */
#define ORACLE_ACT_NONE 0
#define ORACLE_ACT_RELU 1
#define ORACLE_ACT_SILU 2
#define ORACLE_ACT_GELU 3
static double activate(double v, int act) {
  switch (act) {
    case ORACLE_ACT_RELU: return v > 0.0 ? v : 0.0;
    case ORACLE_ACT_SILU: return v / (1.0 + exp(-v));
    case ORACLE_ACT_GELU: return 0.5 * v * (1.0 + erf(v / sqrt(2.0)));
    default: return v;
  }
}

/* r = rows of A / columns of B STORED per slot; r_use <= r = how many of them this slot's adapter has (the
 * paper's future-work "adaptive rank", Sec. 5: a rank per topic; Sec. 4 trains all at one rank, r_use = r).
 * Entries beyond r_use are never read. */
static void lora_token_ex(const void* x, size_t xoff, int xdtype, const void* W, const void* A,
                          const void* B, int wdtype, int64_t slot, int r, int r_use, int act, int64_t d_in,
                          int64_t d_out, double s, double* y /* [d_out] */, double* h /* [r] */);

static void lora_token(const void* x, size_t xoff, int xdtype, const void* W, const void* A,
                       const void* B, int wdtype, int64_t slot, int r, int64_t d_in,
                       int64_t d_out, double s, double* y /* [d_out] */, double* h /* [r] */) {
  lora_token_ex(x, xoff, xdtype, W, A, B, wdtype, slot, r, r, ORACLE_ACT_NONE, d_in, d_out, s, y, h);
}

static void lora_token_ex(const void* x, size_t xoff, int xdtype, const void* W, const void* A,
                          const void* B, int wdtype, int64_t slot, int r, int r_use, int act, int64_t d_in,
                          int64_t d_out, double s, double* y /* [d_out] */, double* h /* [r] */) {
  for (int64_t j = 0; j < d_out; ++j) {
    double acc = 0.0;
    for (int64_t i = 0; i < d_in; ++i)
      acc += ld(W, wdtype, (size_t)(j * d_in + i)) * ld(x, xdtype, xoff + (size_t)i);
    y[j] = acc;
  }
  if (slot < 0 || A == NULL || B == NULL) return;
  for (int p = 0; p < r_use; ++p) {
    double acc = 0.0;
    size_t base = ((size_t)slot * (size_t)r + (size_t)p) * (size_t)d_in;
    for (int64_t i = 0; i < d_in; ++i)
      acc += ld(A, wdtype, base + (size_t)i) * ld(x, xdtype, xoff + (size_t)i);
    h[p] = activate(acc, act);
  }
  for (int64_t j = 0; j < d_out; ++j) {
    double acc = 0.0;
    size_t base = ((size_t)slot * (size_t)d_out + (size_t)j) * (size_t)r;
    for (int p = 0; p < r_use; ++p) acc += ld(B, wdtype, base + (size_t)p) * h[p];
    y[j] += s * acc;
  }
}

static int64_t slot_for(const int32_t* slot_of_expert, int64_t E, int32_t e) {
  if (e < 0 || e >= E || slot_of_expert == NULL) return -1;
  return slot_of_expert[e];
}

/* slot_rank (nullable, [n_slots]): rank of each slot's adapter, at most r; NULL = every slot has rank r.
 * act: ORACLE_ACT_*. */
int moin_oracle_lora_linear_ex(const void* x, const void* W, const void* A, const void* B, int dtype,
                               const int32_t* token_expert, const int32_t* slot_of_expert,
                               const int32_t* slot_rank, int act,
                               int64_t T, int64_t E, int r, int64_t d_in, int64_t d_out, double s,
                               double* y /* [T][d_out] */) {
  if (T < 0 || d_in <= 0 || d_out <= 0 || r < 0 || act < 0 || act > ORACLE_ACT_GELU) return -1;
#pragma omp parallel
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
#pragma omp for schedule(dynamic, 1)
    for (int64_t t = 0; t < T; ++t) {
      int64_t slot = token_expert ? slot_for(slot_of_expert, E, token_expert[t]) : -1;
      int r_use = (slot >= 0 && slot_rank) ? slot_rank[slot] : r;
      if (r_use > r) r_use = r;
      if (r_use < 0) r_use = 0;
      lora_token_ex(x, (size_t)t * (size_t)d_in, dtype, W, A, B, dtype, slot, r, r_use, act, d_in, d_out, s,
                    y + (size_t)t * (size_t)d_out, h);
    }
    free(h);
  }
  return 0;
}

int moin_oracle_lora_linear(const void* x, const void* W, const void* A, const void* B, int dtype,
                            const int32_t* token_expert, const int32_t* slot_of_expert,
                            int64_t T, int64_t E, int r, int64_t d_in, int64_t d_out, double s,
                            double* y /* [T][d_out] */) {
  if (T < 0 || d_in <= 0 || d_out <= 0 || r < 0) return -1;
#pragma omp parallel
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
#pragma omp for schedule(dynamic, 1)
    for (int64_t t = 0; t < T; ++t) {
      int64_t slot = token_expert ? slot_for(slot_of_expert, E, token_expert[t]) : -1;
      lora_token(x, (size_t)t * (size_t)d_in, dtype, W, A, B, dtype, slot, r, d_in, d_out, s,
                 y + (size_t)t * (size_t)d_out, h);
    }
    free(h);
  }
  return 0;
}

/* ------------------------------------------------------------------------------------
 * Decoder forward (Sec. 4: the base model has the Llama-2 architecture; Sec. 3.2: the
 * adapter sits on each linear layer of the network - here the seven projections of every
 * block; Sec. 3.3: one expert per request for the whole forward pass).
 *
 * Conventions (the paper fixes none of them; the GPU library documents the same list):
 *   pre-norm blocks; RMSNorm(v) = v / sqrt(mean(v^2) + eps) * gain;
 *   rotary embedding with the half-split pairing (i, i + head_dim/2), angle
 *   pos * base^(-2i/head_dim), positions restart at 0 in every request;
 *   causal softmax attention inside each request only, scale 1/sqrt(head_dim);
 *   grouped-query attention: query head h reads kv head h / (n_heads / n_kv_heads);
 *   MLP: down( silu(gate(v)) * up(v) ); no biases; untied lm_head; no adapter on
 *   embedding or lm_head.
 *
 * round_storage != 0 rounds to bf16 wherever the GPU library stores a tensor in bf16
 * (norm outputs, projection outputs, rotated q/k, attention output, SwiGLU output,
 * logits) and where it documents a bf16 tensor-core operand that is never stored (the
 * un-normalised attention weights exp(s - max)); the residual stream stays unrounded (the
 * library keeps it in fp32).
 * ------------------------------------------------------------------------------------ */
typedef struct {
  int32_t n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, E, r, n_slots;
  double rms_eps, rope_base, scale;
  const uint16_t* embed;      /* [vocab][hidden] bf16 */
  const uint16_t* lm_head;    /* [vocab][hidden] bf16 */
  const uint16_t* final_norm; /* [hidden] */
  const uint16_t* const* attn_norm; /* [n_layers] -> [hidden] */
  const uint16_t* const* mlp_norm;  /* [n_layers] -> [hidden] */
  const uint16_t* const* W;   /* [n_layers*7] -> [d_out][d_in], order q,k,v,o,gate,up,down */
  const uint16_t* const* A;   /* [n_layers*7] -> [n_slots][r][d_in], may be NULL entries */
  const uint16_t* const* B;   /* [n_layers*7] -> [n_slots][d_out][r] */
  const int32_t* slot_of_expert; /* [E] */
} moin_oracle_model;

static double maybe_round(double v, int on) { return on ? round_bf16(v) : v; }

static void rmsnorm(const double* v, const uint16_t* gain, int n, double eps, int rnd, double* out) {
  double ss = 0.0;
  for (int i = 0; i < n; ++i) ss += v[i] * v[i];
  double inv = 1.0 / sqrt(ss / (double)n + eps);
  for (int i = 0; i < n; ++i) out[i] = maybe_round(v[i] * inv * ld(gain, ORACLE_BF16, (size_t)i), rnd);
}

/* One projection of one request: rows [0, L) of in[L][d_in] -> out[L][d_out]; slots[t] = adapter slot of
 * token t (-1: base only).  The paper uses one expert per request (Sec. 3.3: slots all equal); an expert per
 * token is its future-work variant (Sec. 5) and needs nothing but a slot per row. */
static void project(const moin_oracle_model* m, int layer, int proj, const double* in, int64_t L,
                    int64_t d_in, int64_t d_out, const int64_t* slots, int rnd, double* out, double* h) {
  const void* W = m->W[layer * 7 + proj];
  const void* A = m->A ? m->A[layer * 7 + proj] : NULL;
  const void* B = m->B ? m->B[layer * 7 + proj] : NULL;
  for (int64_t t = 0; t < L; ++t) {
    /* activations are doubles here; weights are bf16 */
    double* y = out + (size_t)t * (size_t)d_out;
    lora_token(in, (size_t)t * (size_t)d_in, ORACLE_F64, W, A, B, ORACLE_BF16, slots[t], m->r, d_in,
               d_out, m->scale, y, h);
    if (rnd)
      for (int64_t j = 0; j < d_out; ++j) y[j] = round_bf16(y[j]);
  }
}

static void rope_inplace(double* v /* [L][n_h*hd] */, int64_t L, int n_h, int hd, double base, int rnd) {
  int half = hd / 2;
  for (int64_t t = 0; t < L; ++t)
    for (int h = 0; h < n_h; ++h) {
      double* p = v + ((size_t)t * (size_t)n_h + (size_t)h) * (size_t)hd;
      for (int i = 0; i < half; ++i) {
        double ang = (double)t * pow(base, -2.0 * (double)i / (double)hd);
        double c = cos(ang), s = sin(ang);
        double a = p[i], b = p[i + half];
        p[i] = maybe_round(a * c - b * s, rnd);
        p[i + half] = maybe_round(b * c + a * s, rnd);
      }
    }
}

/* Blocks [layer_begin, layer_end) applied to one request's residual stream xr[L][hidden]. */
static int run_blocks(const moin_oracle_model* m, int layer_begin, int layer_end, double* xr,
                      int64_t L, const int64_t* slot, int rnd) {
  const int H = m->hidden, nh = m->n_heads, nkv = m->n_kv_heads, hd = m->head_dim, F = m->ffn;
  const int qd = nh * hd, kvd = nkv * hd, group = nh / nkv;
  size_t LL = (size_t)L;
  double* xn = (double*)malloc(sizeof(double) * LL * (size_t)H);
  double* q = (double*)malloc(sizeof(double) * LL * (size_t)qd);
  double* k = (double*)malloc(sizeof(double) * LL * (size_t)kvd);
  double* v = (double*)malloc(sizeof(double) * LL * (size_t)kvd);
  double* att = (double*)malloc(sizeof(double) * LL * (size_t)qd);
  double* o = (double*)malloc(sizeof(double) * LL * (size_t)H);
  double* gate = (double*)malloc(sizeof(double) * LL * (size_t)F);
  double* up = (double*)malloc(sizeof(double) * LL * (size_t)F);
  double* prob = (double*)malloc(sizeof(double) * LL);
  double* h = (double*)malloc(sizeof(double) * (size_t)(m->r > 0 ? m->r : 1));
  if (!xn || !q || !k || !v || !att || !o || !gate || !up || !prob || !h) return -2;
  double sm_scale = 1.0 / sqrt((double)hd);
  for (int l = layer_begin; l < layer_end; ++l) {
    for (int64_t t = 0; t < L; ++t)
      rmsnorm(xr + (size_t)t * H, m->attn_norm[l], H, m->rms_eps, rnd, xn + (size_t)t * H);
    project(m, l, 0, xn, L, H, qd, slot, rnd, q, h);
    project(m, l, 1, xn, L, H, kvd, slot, rnd, k, h);
    project(m, l, 2, xn, L, H, kvd, slot, rnd, v, h);
    rope_inplace(q, L, nh, hd, m->rope_base, rnd);
    rope_inplace(k, L, nkv, hd, m->rope_base, rnd);
    for (int64_t t = 0; t < L; ++t)
      for (int hq = 0; hq < nh; ++hq) {
        int hk = hq / group;
        const double* qv = q + ((size_t)t * nh + hq) * hd;
        double mx = -INFINITY;
        for (int64_t u = 0; u <= t; ++u) {
          const double* kv = k + ((size_t)u * nkv + hk) * hd;
          double s = 0.0;
          for (int i = 0; i < hd; ++i) s += qv[i] * kv[i];
          prob[u] = s * sm_scale;
          if (prob[u] > mx) mx = prob[u];
        }
        double den = 0.0;
        for (int64_t u = 0; u <= t; ++u) {
          prob[u] = exp(prob[u] - mx);
          den += prob[u];                          /* normaliser: sum of the unrounded weights */
          prob[u] = maybe_round(prob[u], rnd);     /* storage-rounded variant: the library feeds the weights to the
                                                      tensor cores as bf16 (the one operand rounding that is not a
                                                      stored tensor); the exact variant keeps them in double */
        }
        double* ov = att + ((size_t)t * nh + hq) * hd;
        for (int i = 0; i < hd; ++i) {
          double acc = 0.0;
          for (int64_t u = 0; u <= t; ++u) acc += prob[u] * v[((size_t)u * nkv + hk) * hd + i];
          ov[i] = maybe_round(acc / den, rnd);
        }
      }
    project(m, l, 3, att, L, qd, H, slot, rnd, o, h);
    for (size_t i = 0; i < LL * (size_t)H; ++i) xr[i] += o[i];
    for (int64_t t = 0; t < L; ++t)
      rmsnorm(xr + (size_t)t * H, m->mlp_norm[l], H, m->rms_eps, rnd, xn + (size_t)t * H);
    project(m, l, 4, xn, L, H, F, slot, rnd, gate, h);
    project(m, l, 5, xn, L, H, F, slot, rnd, up, h);
    for (size_t i = 0; i < LL * (size_t)F; ++i) {
      double g = gate[i];
      gate[i] = maybe_round(g / (1.0 + exp(-g)) * up[i], rnd);
    }
    project(m, l, 6, gate, L, F, H, slot, rnd, o, h);
    for (size_t i = 0; i < LL * (size_t)H; ++i) xr[i] += o[i];
  }
  free(xn); free(q); free(k); free(v); free(att); free(o); free(gate); free(up); free(prob); free(h);
  return 0;
}

/* Full or partial forward.
 *   hidden_in  (nullable) [T][hidden] double: start from this residual stream instead of the
 *              embedding lookup (used to feed one block at a time);
 *   layers [layer_begin, layer_end) are applied;
 *   hidden_out (nullable) [T][hidden] double: residual stream after layer_end-1;
 *   logits     (nullable) [T][vocab] double: final norm + lm_head (only meaningful when
 *              layer_end == n_layers). */
int moin_oracle_decoder_forward(const moin_oracle_model* m, const int32_t* tokens,
                                const int32_t* cu_seqlens, const int32_t* req_expert,
                                const int32_t* token_expert, int32_t R,
                                int64_t T, int layer_begin, int layer_end, int round_storage,
                                const double* hidden_in, double* hidden_out, double* logits) {
  if (!m || R < 0 || T < 0 || layer_begin < 0 || layer_end > m->n_layers || layer_begin > layer_end)
    return -1;
  const int H = m->hidden;
  int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t rq = 0; rq < R; ++rq) {
    int64_t t0 = cu_seqlens[rq], L = cu_seqlens[rq + 1] - cu_seqlens[rq];
    if (L <= 0) continue;
    /* adapter slot of every token: the request's expert (Sec. 3.3), or the token's own if token_expert is given */
    int64_t* slot = (int64_t*)malloc(sizeof(int64_t) * (size_t)L);
    double* xr = (double*)malloc(sizeof(double) * (size_t)L * (size_t)H);
    if (!xr || !slot) { rc = -2; free(xr); free(slot); continue; }
    for (int64_t t = 0; t < L; ++t) {
      if (token_expert) slot[t] = slot_for(m->slot_of_expert, m->E, token_expert[t0 + t]);
      else slot[t] = req_expert ? slot_for(m->slot_of_expert, m->E, req_expert[rq]) : -1;
    }
    for (int64_t t = 0; t < L; ++t)
      for (int i = 0; i < H; ++i)
        xr[(size_t)t * H + i] = hidden_in ? hidden_in[(size_t)(t0 + t) * H + i]
                                          : ld(m->embed, ORACLE_BF16, (size_t)tokens[t0 + t] * H + i);
    int e = run_blocks(m, layer_begin, layer_end, xr, L, slot, round_storage);
    if (e) rc = e;
    if (hidden_out) memcpy(hidden_out + (size_t)t0 * H, xr, sizeof(double) * (size_t)L * (size_t)H);
    if (logits) {
      double* xn = (double*)malloc(sizeof(double) * (size_t)H);
      for (int64_t t = 0; t < L; ++t) {
        rmsnorm(xr + (size_t)t * H, m->final_norm, H, m->rms_eps, round_storage, xn);
        double* out = logits + (size_t)(t0 + t) * (size_t)m->vocab;
        for (int j = 0; j < m->vocab; ++j) {
          double acc = 0.0;
          for (int i = 0; i < H; ++i) acc += ld(m->lm_head, ORACLE_BF16, (size_t)j * H + i) * xn[i];
          out[j] = maybe_round(acc, round_storage);
        }
      }
      free(xn);
    }
    free(xr);
    free(slot);
  }
  return rc;
}

/* ------------------------------------------------------------------------------------
 * Grouping of tokens by adapter slot (what a multi-adapter batch needs before it can
 * stream each adapter once; the paper only names the need, Sec. 1).  Plain definition:
 * a stable sort of token indices by slot, tokens without an adapter last.
 *   perm[T]          token indices, ordered by (slot, token index), slot -1 at the end
 *   seg_slot[S], seg_start[S+1]  one segment per distinct slot >= 0, ascending slot
 * Returns S (number of segments) or a negative error.
 * ------------------------------------------------------------------------------------ */
int64_t moin_oracle_bucket(const int32_t* token_expert, const int32_t* slot_of_expert, int64_t T,
                           int64_t E, int64_t n_slots, int32_t* perm, int32_t* seg_slot,
                           int32_t* seg_start) {
  if (T < 0 || n_slots < 0) return -1;
  int64_t pos = 0, S = 0;
  for (int64_t s = 0; s < n_slots; ++s) {
    int64_t first = pos;
    for (int64_t t = 0; t < T; ++t)
      if (slot_for(slot_of_expert, E, token_expert[t]) == s) perm[pos++] = (int32_t)t;
    if (pos > first) {
      seg_slot[S] = (int32_t)s;
      seg_start[S] = (int32_t)first;
      ++S;
    }
  }
  seg_start[S] = (int32_t)pos;
  for (int64_t t = 0; t < T; ++t) {
    int64_t s = slot_for(slot_of_expert, E, token_expert[t]);
    if (s < 0 || s >= n_slots) perm[pos++] = (int32_t)t;
  }
  return S;
}

/* ---------------------------------------------------------------------------------------
 * K-means update (Sec. 3.1: K-means directly in the document embedding space; Sec. 4: the
 * cluster centroid is the topic embedding).  Given the assignment of every point, centroid
 * k becomes the arithmetic mean of its members, summed in increasing point order.
 * Readings: a cluster without members keeps its previous centroid; assignments outside
 * [0, K) are ignored.  The assignment step itself is the router above (nearest centroid
 * under the cosine metric), so one Lloyd iteration = route, then this.
 *
 * x [N, D], c_old [K, D] (double or bf16 bits); assign [N]; c_new [K, D] double; counts [K].
 * ------------------------------------------------------------------------------------ */
int moin_oracle_kmeans_update(const void* x, const void* c_old, int dtype, const int32_t* assign,
                              int64_t N, int64_t K, int64_t D, double* c_new, int64_t* counts) {
  if (N < 0 || K < 1 || D < 1) return -1;
  for (int64_t k = 0; k < K; ++k) counts[k] = 0;
  for (int64_t i = 0; i < K * D; ++i) c_new[i] = 0.0;
  for (int64_t i = 0; i < N; ++i) {
    const int64_t k = assign[i];
    if (k < 0 || k >= K) continue;
    counts[k] += 1;
    for (int64_t d = 0; d < D; ++d) c_new[k * D + d] += ld(x, dtype, (size_t)(i * D + d));
  }
  for (int64_t k = 0; k < K; ++k)
    for (int64_t d = 0; d < D; ++d) {
      if (counts[k] > 0) c_new[k * D + d] /= (double)counts[k];
      else c_new[k * D + d] = ld(c_old, dtype, (size_t)(k * D + d));
    }
  return 0;
}

/* ------------------------------------------------------------------------------------
 * Quantised frozen base weights (Sec. 5 lists a quantised base model with the adapters kept
 * in 16 bits, "QLoRA-like", as a variant; it fixes no format).  Format taken here: one byte per
 * weight in the 8-bit floating-point format with 4 exponent and 3 mantissa bits, exponent
 * bias 7, no infinities (exponent 15 with mantissa 7 is NaN, largest finite value 448), plus
 * one fp32 scale per output row.  The weight the layer uses is
 *     W[j][i] = bf16( fp32( value(code[j][i]) * scale[j] ) ),
 * i.e. the code's value times the row scale, multiplied in fp32 and rounded once more to the
 * bf16 the GEMMs read.  Everything after that is the ordinary layer on W.
 * ------------------------------------------------------------------------------------ */
static float e4m3_value(uint8_t c) {
  int sign = c >> 7, ex = (c >> 3) & 15, man = c & 7;
  float v;
  if (ex == 15 && man == 7) return NAN;
  if (ex == 0) v = ldexpf((float)man, -9);                 /* subnormal: man / 8 * 2^-6 */
  else v = ldexpf(1.0f + (float)man / 8.0f, ex - 7);
  return sign ? -v : v;
}

double moin_oracle_e4m3_value(int code) { return (double)e4m3_value((uint8_t)code); }

int moin_oracle_dequant_fp8(const uint8_t* codes, const float* scale, int64_t d_out, int64_t d_in,
                            uint16_t* out_bf16 /* [d_out][d_in] bf16 bit patterns */) {
  if (!codes || !scale || !out_bf16 || d_out < 0 || d_in < 0) return -1;
  for (int64_t j = 0; j < d_out; ++j)
    for (int64_t i = 0; i < d_in; ++i) {
      volatile float prod = e4m3_value(codes[j * d_in + i]) * scale[j];   /* fp32 product, rounded to fp32 */
      double r = round_bf16((double)prod);
      float f = (float)r;                                                  /* exact: r is a bf16 value */
      uint32_t u;
      memcpy(&u, &f, 4);
      out_bf16[j * d_in + i] = (uint16_t)(u >> 16);
    }
  return 0;
}
