/*
 * spkv_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision CPU statement of what Self-Pruned KV
 * attention (SP-KV) computes at inference time.  It exists to check the CUDA
 * library; it shares no code with it and nothing in the product path may call
 * it.  Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Two independent formulations of the same definition live here (and, after them, the
 * soft-gated whole-sequence forward of the paper's training section, Eq. 6-7):
 *
 *   "mask form"      (orcB_*)  Eq. 2-5 of the paper written out literally:
 *                    threshold every position, build the additive bias
 *                    B[t][s] = M_causal + g over ALL positions s in [0,T),
 *                    softmax the biased scores, weight the values.
 *
 *   "streaming form" (orcA_*)  the cache state machine of the paper's
 *                    inference description (Appendix "Inference Kernels"):
 *                    a ring of the w most recent pairs plus an append-only
 *                    list of pairs that passed the threshold when they aged
 *                    out of the ring; attention is a dense softmax over
 *                    ring U kept list.
 *
 * The two never call one another or a common attention helper, so their
 * agreement at every position (tests) is a brute-force pin.
 *
 * Conventions (readings of the paper where it is silent are listed in the
 * design notes of the repository):
 *   - storage values are bfloat16 bit patterns (uint16_t), widened exactly to
 *     double; every sum, exponential and division is done in double;
 *   - the keep decision is taken on the float32 logit: keep <=> logit >= tau_logit,
 *     tau_logit = (float) log(tau / (1 - tau))   (Eq. 1-2; sigma is monotone);
 *   - window of query t = positions s with 0 <= t - s < w, t itself included;
 *   - query head j of a group reads KV head floor(j / G).
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py
 * (closed forms, limiting cases tau = -inf / +inf / w >= T, mask form ==
 * streaming form, enumeration of the visible set with one-hot values, kept-set
 * identity).  No function is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ helpers */

/* bfloat16 -> double: the 16 bits are the top half of an IEEE float32. */
static double bf16_widen(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

double orc_bf16_to_double(uint16_t h) { return bf16_widen(h); }

/* Eq. 1: logistic sigmoid. */
double orc_sigmoid(double z) { return 1.0 / (1.0 + exp(-z)); }

/* Threshold moved to logit space: u >= tau  <=>  logit >= log(tau/(1-tau)).
 * tau <= 0 keeps everything (-inf); tau >= 1 keeps nothing (+inf), since u lies
 * in the open interval (0,1) (Eq. 1). */
float orc_tau_logit(double tau) {
  if (!(tau > 0.0)) return -INFINITY;
  if (!(tau < 1.0)) return INFINITY;
  return (float)log(tau / (1.0 - tau));
}

/* ------------------------------------------------------------ Eq. 1: scores */

/* Linear predictor variant: logit[n][h] = <W[h], x[n]> + b[h]. */
void orc_score_linear(const uint16_t *x, int n_tok, int d_in, const uint16_t *W,
                      const float *b, int n_kv_heads, double *logit_out) {
  for (int n = 0; n < n_tok; ++n)
    for (int h = 0; h < n_kv_heads; ++h) {
      double acc = 0.0;
      for (int i = 0; i < d_in; ++i)
        acc += bf16_widen(W[(size_t)h * d_in + i]) * bf16_widen(x[(size_t)n * d_in + i]);
      logit_out[(size_t)n * n_kv_heads + h] = acc + (double)b[h];
    }
}

/* Two-layer perceptron of the paper's listing:
 * logit = W2 . SiLU(W1 x + b1) + b2, SiLU(z) = z * sigmoid(z);
 * first layer shared by the KV heads of a layer, one output per KV head. */
void orc_score_mlp(const uint16_t *x, int n_tok, int d_in, const uint16_t *W1,
                   const float *b1, int hidden, const uint16_t *W2, const float *b2,
                   int n_kv_heads, double *logit_out) {
  double *a = (double *)malloc(sizeof(double) * (size_t)hidden);
  for (int n = 0; n < n_tok; ++n) {
    for (int j = 0; j < hidden; ++j) {
      double z = (double)b1[j];
      for (int i = 0; i < d_in; ++i)
        z += bf16_widen(W1[(size_t)j * d_in + i]) * bf16_widen(x[(size_t)n * d_in + i]);
      a[j] = z * orc_sigmoid(z);
    }
    for (int h = 0; h < n_kv_heads; ++h) {
      double acc = (double)b2[h];
      for (int j = 0; j < hidden; ++j) acc += bf16_widen(W2[(size_t)h * hidden + j]) * a[j];
      logit_out[(size_t)n * n_kv_heads + h] = acc;
    }
  }
  free(a);
}

/* ------------------------------------------------- mask form (Eq. 2 - Eq. 5) */

/*
 * One query position t of one KV head over a full, uncompressed sequence.
 *   K, V   [T][D] bf16   all keys / values, positions 0..T-1
 *   logit  [T]   float   utility logits
 *   q      [G][D] bf16   the G query heads of the group at position t
 *   out    [G][D] double; lse [G] double or NULL (natural-log sum-exp of the
 *          biased, scaled scores)
 * Every position s in [0,T) gets a bias: 0 when causal and (gated on or inside
 * the window), -inf otherwise; the softmax runs over the whole row.
 */
void orcB_attend_row_sinks(const uint16_t *K, const uint16_t *V, const float *logit, int T,
                           int t, int w, float tau_logit, int n_sink, const uint16_t *q, int G,
                           int D, double scale, double *out, double *lse) {
  double *score = (double *)malloc(sizeof(double) * (size_t)T);
  for (int g = 0; g < G; ++g) {
    double mx = -INFINITY;
    for (int s = 0; s < T; ++s) {
      int z = (logit[s] >= tau_logit) ? 1 : 0;                 /* Eq. 2 */
      int in_win = (t - s >= 0) && (t - s < w);                /* window indicator */
      int sink = s < n_sink;     /* "Fixed Attention Sinks" variant: the first n_sink
                                    positions are retained whatever their gate says */
      double gate = (z || in_win || sink) ? 0.0 : -INFINITY;   /* Eq. 3 */
      double causal = (s <= t) ? 0.0 : -INFINITY;
      double bias = causal + gate;                             /* Eq. 4 */
      double dot = 0.0;
      for (int i = 0; i < D; ++i)
        dot += bf16_widen(q[(size_t)g * D + i]) * bf16_widen(K[(size_t)s * D + i]);
      score[s] = dot * scale + bias;
      if (score[s] > mx) mx = score[s];
    }
    double denom = 0.0;
    for (int s = 0; s < T; ++s) denom += exp(score[s] - mx);   /* exp(-inf) = 0 */
    for (int i = 0; i < D; ++i) out[(size_t)g * D + i] = 0.0;
    for (int s = 0; s < T; ++s) {
      double p = exp(score[s] - mx) / denom;                   /* Eq. 5 */
      if (p == 0.0) continue;
      for (int i = 0; i < D; ++i) out[(size_t)g * D + i] += p * bf16_widen(V[(size_t)s * D + i]);
    }
    if (lse) lse[g] = mx + log(denom);
  }
  free(score);
}

/* The method as the paper defines it (no sink tokens). */
void orcB_attend_row(const uint16_t *K, const uint16_t *V, const float *logit, int T,
                     int t, int w, float tau_logit, const uint16_t *q, int G, int D,
                     double scale, double *out, double *lse) {
  orcB_attend_row_sinks(K, V, logit, T, t, w, tau_logit, 0, q, G, D, scale, out, lse);
}

/* Whole-sequence mask form: out[t][g][:] for every t (O(T^2); tiny T only). */
void orcB_attend_all_sinks(const uint16_t *K, const uint16_t *V, const float *logit, int T,
                           int w, float tau_logit, int n_sink, const uint16_t *q /*[T][G][D]*/,
                           int G, int D, double scale, double *out /*[T][G][D]*/) {
  for (int t = 0; t < T; ++t)
    orcB_attend_row_sinks(K, V, logit, T, t, w, tau_logit, n_sink, q + (size_t)t * G * D, G, D,
                          scale, out + (size_t)t * G * D, NULL);
}

void orcB_attend_all(const uint16_t *K, const uint16_t *V, const float *logit, int T,
                     int w, float tau_logit, const uint16_t *q /*[T][G][D]*/, int G, int D,
                     double scale, double *out /*[T][G][D]*/) {
  orcB_attend_all_sinks(K, V, logit, T, w, tau_logit, 0, q, G, D, scale, out);
}

/* ------------------------------ soft-gated forward (Eq. 6 and Eq. 7: the training-time form) */

/*
 * Gate of one position.  u = sigma(logit) (Eq. 1).  During the annealed switch to hard gating the
 * paper interpolates u~ = (1 - alpha) u + alpha 1[u >= tau] (Eq. 7): alpha = 0 is soft gating,
 * alpha = 1 the binary gate.  The threshold is applied as everywhere else, on the float32 logit.
 * Returns the additive bias log u~ (Eq. 6 with u~ for u); -inf when u~ = 0.
 * For alpha = 0 the logarithm of the sigmoid is taken without forming the sigmoid:
 * log sigma(l) = -log(1 + e^-l), finite for every finite l.  (The epsilon the paper's listing
 * adds inside the logarithm is a guard for gradients; it is not part of Eq. 6 and not here.)
 */
double orc_gate_log_bias(float logit, double alpha, float tau_logit) {
  double l = (double)logit;
  if (alpha == 0.0) return l >= 0.0 ? -log1p(exp(-l)) : l - log1p(exp(l));
  double u = orc_sigmoid(l);
  double z = (logit >= tau_logit) ? 1.0 : 0.0;                 /* Eq. 2 */
  double u_tilde = (1.0 - alpha) * u + alpha * z;              /* Eq. 7 */
  return log(u_tilde);                                         /* log(0) = -inf */
}

/*
 * Soft-gated attention for one query position t of one KV head over the whole sequence:
 * the bias of Eq. 4 with the binary gate replaced by log u~_s (Eq. 6).  Three regions of a row:
 * the window 0 <= t - s < w has bias 0 whatever the gate; an earlier position has bias
 * log u~_s; a future position -inf.  Arguments as orcB_attend_row; alpha as above.
 */
void orcB_attend_row_soft(const uint16_t *K, const uint16_t *V, const float *logit, int T,
                          int t, int w, double alpha, float tau_logit, const uint16_t *q, int G,
                          int D, double scale, double *out, double *lse) {
  double *a = (double *)malloc(sizeof(double) * (size_t)T);   /* biased, scaled scores of the row */
  for (int g = 0; g < G; ++g) {
    const uint16_t *qg = q + (size_t)g * D;
    double top = -INFINITY;
    for (int s = 0; s < T; ++s) {
      double bias_ts;
      if (s > t) bias_ts = -INFINITY;                                      /* future          */
      else if (t - s < w) bias_ts = 0.0;                                   /* sliding window  */
      else bias_ts = orc_gate_log_bias(logit[s], alpha, tau_logit);        /* long range: log u~_s */
      double qk = 0.0;
      for (int i = 0; i < D; ++i) qk += bf16_widen(qg[i]) * bf16_widen(K[(size_t)s * D + i]);
      a[s] = qk * scale + bias_ts;
      if (a[s] > top) top = a[s];
    }
    double z_row = 0.0;
    for (int s = 0; s < T; ++s) z_row += exp(a[s] - top);
    for (int i = 0; i < D; ++i) out[(size_t)g * D + i] = 0.0;
    for (int s = 0; s < T; ++s) {
      double weight = exp(a[s] - top) / z_row;
      if (weight == 0.0) continue;
      for (int i = 0; i < D; ++i) out[(size_t)g * D + i] += weight * bf16_widen(V[(size_t)s * D + i]);
    }
    if (lse) lse[g] = top + log(z_row);
  }
  free(a);
}

/* Soft-gated forward for every position (O(T^2)), rows in parallel. */
void orcB_attend_all_soft(const uint16_t *K, const uint16_t *V, const float *logit, int T, int w,
                          double alpha, float tau_logit, const uint16_t *q /*[T][G][D]*/, int G,
                          int D, double scale, double *out /*[T][G][D]*/, double *lse /*[T][G] or NULL*/) {
#pragma omp parallel for schedule(dynamic, 8)
  for (int t = 0; t < T; ++t)
    orcB_attend_row_soft(K, V, logit, T, t, w, alpha, tau_logit, q + (size_t)t * G * D, G, D, scale,
                         out + (size_t)t * G * D, lse ? lse + (size_t)t * G : NULL);
}

/* Eq. 8 gate density over one (layer, head): mean of z over all T positions,
 * and the cache-centric variant (kept pairs / pairs that left the window). */
void orcB_density(const float *logit, int T, int w, float tau_logit, double *rho_all,
                  double *rho_cache) {
  long z_all = 0, z_out = 0;
  for (int s = 0; s < T; ++s) {
    int z = logit[s] >= tau_logit;
    z_all += z;
    if (s <= T - 1 - w) z_out += z; /* positions outside the window of the last query */
  }
  *rho_all = T > 0 ? (double)z_all / T : 0.0;
  *rho_cache = (T - w) > 0 ? (double)z_out / (T - w) : 0.0;
}

/* -------------------------------------------------- streaming form (state) */

typedef struct orcA_unit {
  int w, D;
  int n_sink;        /* positions < n_sink are kept whatever their logit (0: none) */
  long t;            /* number of pairs appended so far = next position        */
  uint16_t *ring_k;  /* [w][D]  slot (s mod w) holds position s                 */
  uint16_t *ring_v;
  float *ring_logit; /* [w]                                                     */
  long n_kept, cap;  /* append-only kept list                                   */
  int32_t *kept_pos;
  uint16_t *kept_k, *kept_v;
} orcA_unit;

orcA_unit *orcA_new(int w, int D) {
  orcA_unit *u = (orcA_unit *)calloc(1, sizeof *u);
  u->w = w;
  u->D = D;
  u->ring_k = (uint16_t *)calloc((size_t)w * D, 2);
  u->ring_v = (uint16_t *)calloc((size_t)w * D, 2);
  u->ring_logit = (float *)calloc((size_t)w, sizeof(float));
  return u;
}

void orcA_set_sinks(orcA_unit *u, int n_sink) { u->n_sink = n_sink; }

void orcA_free(orcA_unit *u) {
  if (!u) return;
  free(u->ring_k); free(u->ring_v); free(u->ring_logit);
  free(u->kept_pos); free(u->kept_k); free(u->kept_v);
  free(u);
}

static void orcA_keep(orcA_unit *u, long pos, const uint16_t *k, const uint16_t *v) {
  if (u->n_kept == u->cap) {
    u->cap = u->cap ? 2 * u->cap : 256;
    u->kept_pos = (int32_t *)realloc(u->kept_pos, sizeof(int32_t) * (size_t)u->cap);
    u->kept_k = (uint16_t *)realloc(u->kept_k, 2 * (size_t)u->cap * u->D);
    u->kept_v = (uint16_t *)realloc(u->kept_v, 2 * (size_t)u->cap * u->D);
  }
  u->kept_pos[u->n_kept] = (int32_t)pos;
  memcpy(u->kept_k + (size_t)u->n_kept * u->D, k, 2 * (size_t)u->D);
  memcpy(u->kept_v + (size_t)u->n_kept * u->D, v, 2 * (size_t)u->D);
  u->n_kept++;
}

/* Append the pair of position t.  When the ring is full, the pair of position
 * t - w leaves it: it joins the kept list iff its stored logit >= tau_logit
 * (threshold applied at window exit, with the threshold current at that time)
 * or it is one of the first n_sink positions (sink-token variant); otherwise it
 * is gone for good. */
void orcA_append(orcA_unit *u, const uint16_t *k, const uint16_t *v, float logit,
                 float tau_logit) {
  long slot = u->t % u->w;
  if (u->t >= u->w) {
    if (u->ring_logit[slot] >= tau_logit || u->t - u->w < u->n_sink)
      orcA_keep(u, u->t - u->w, u->ring_k + (size_t)slot * u->D, u->ring_v + (size_t)slot * u->D);
  }
  memcpy(u->ring_k + (size_t)slot * u->D, k, 2 * (size_t)u->D);
  memcpy(u->ring_v + (size_t)slot * u->D, v, 2 * (size_t)u->D);
  u->ring_logit[slot] = logit;
  u->t++;
}

/* Dense softmax attention of the group's G query heads over ring U kept list,
 * for the query whose own pair was appended last (position t-1). */
void orcA_attend(const orcA_unit *u, const uint16_t *q, int G, double scale, double *out,
                 double *lse) {
  const int D = u->D;
  long n_ring = u->t < u->w ? u->t : u->w;
  long n = n_ring + u->n_kept;
  double *p = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
  for (int g = 0; g < G; ++g) {
    double mx = -INFINITY;
    for (long j = 0; j < n; ++j) {
      const uint16_t *kr = j < u->n_kept ? u->kept_k + (size_t)j * D
                                         : u->ring_k + (size_t)(j - u->n_kept) * D;
      double dot = 0.0;
      for (int i = 0; i < D; ++i) dot += bf16_widen(q[(size_t)g * D + i]) * bf16_widen(kr[i]);
      p[j] = dot * scale;
      if (p[j] > mx) mx = p[j];
    }
    double denom = 0.0;
    for (long j = 0; j < n; ++j) { p[j] = exp(p[j] - mx); denom += p[j]; }
    for (int i = 0; i < D; ++i) out[(size_t)g * D + i] = 0.0;
    for (long j = 0; j < n; ++j) {
      const uint16_t *vr = j < u->n_kept ? u->kept_v + (size_t)j * D
                                         : u->ring_v + (size_t)(j - u->n_kept) * D;
      double pj = p[j] / denom;
      for (int i = 0; i < D; ++i) out[(size_t)g * D + i] += pj * bf16_widen(vr[i]);
    }
    if (lse) lse[g] = n > 0 ? mx + log(denom) : -INFINITY;
  }
  free(p);
}

/* Chunked prefill by definition: C times (append, attend).  q/out may be NULL
 * to build state only. */
void orcA_prefill(orcA_unit *u, int C, const uint16_t *k /*[C][D]*/, const uint16_t *v,
                  const float *logit /*[C]*/, float tau_logit, const uint16_t *q /*[C][G][D]*/,
                  int G, double scale, double *out /*[C][G][D]*/) {
  for (int i = 0; i < C; ++i) {
    orcA_append(u, k + (size_t)i * u->D, v + (size_t)i * u->D, logit[i], tau_logit);
    if (q && out)
      orcA_attend(u, q + (size_t)i * G * u->D, G, scale, out + (size_t)i * G * u->D, NULL);
  }
}

long orcA_t(const orcA_unit *u) { return u->t; }
long orcA_len(const orcA_unit *u) { return u->n_kept; }

void orcA_get_kept(const orcA_unit *u, int32_t *pos, uint16_t *k, uint16_t *v) {
  if (pos) memcpy(pos, u->kept_pos, sizeof(int32_t) * (size_t)u->n_kept);
  if (k) memcpy(k, u->kept_k, 2 * (size_t)u->n_kept * u->D);
  if (v) memcpy(v, u->kept_v, 2 * (size_t)u->n_kept * u->D);
}

/* Ring contents in ascending position order: positions max(0,t-w) .. t-1. */
void orcA_get_window(const orcA_unit *u, int32_t *pos, uint16_t *k, uint16_t *v, float *logit) {
  long n = u->t < u->w ? u->t : u->w;
  long first = u->t - n;
  for (long j = 0; j < n; ++j) {
    long s = first + j, slot = s % u->w;
    if (pos) pos[j] = (int32_t)s;
    if (k) memcpy(k + (size_t)j * u->D, u->ring_k + (size_t)slot * u->D, 2 * (size_t)u->D);
    if (v) memcpy(v + (size_t)j * u->D, u->ring_v + (size_t)slot * u->D, 2 * (size_t)u->D);
    if (logit) logit[j] = u->ring_logit[slot];
  }
}

/* One decode step for many independent units (the unit loop is the only thing
 * run in parallel; used by the benchmark's CPU-baseline leg and by tests). */
void orcA_step_batch(orcA_unit **units, int n_units, const uint16_t *k /*[n][D]*/,
                     const uint16_t *v, const float *logit /*[n]*/, float tau_logit,
                     const uint16_t *q /*[n][G][D]*/, int G, double scale,
                     double *out /*[n][G][D]*/) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int i = 0; i < n_units; ++i) {
    const int D = units[i]->D;
    orcA_append(units[i], k + (size_t)i * D, v + (size_t)i * D, logit[i], tau_logit);
    orcA_attend(units[i], q + (size_t)i * G * D, G, scale, out + (size_t)i * G * D, NULL);
  }
}

/* State build for many units at once: unit i receives n pairs. */
void orcA_prefill_batch(orcA_unit **units, int n_units, int C, const uint16_t *k /*[n][C][D]*/,
                        const uint16_t *v, const float *logit /*[n][C]*/, float tau_logit) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int i = 0; i < n_units; ++i) {
    const int D = units[i]->D;
    orcA_prefill(units[i], C, k + (size_t)i * C * D, v + (size_t)i * C * D,
                 logit + (size_t)i * C, tau_logit, NULL, 0, 0.0, NULL);
  }
}

#ifdef _OPENMP
#include <omp.h>
int orc_threads(void) { return omp_get_max_threads(); }
#else
int orc_threads(void) { return 1; }
#endif
