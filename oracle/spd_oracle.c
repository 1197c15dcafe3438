/*
 * CPU oracle for Superposed Decoding (SPD).  TEST INFRASTRUCTURE ONLY: it exists to check
 * the CUDA library and to be timed as a CPU baseline.  It is deliberately plain and slow, it
 * shares no code with the CUDA path, and no product code may call it.
 *
 * What it follows (Shen et al., "Superposed Decoding", Sections 3, 3.1, 3.2, Algorithm 1,
 * Appendix B):
 *   - first timestep: one dense causal pass over the prefix; draft i takes the i-th most
 *     probable token and its probability (Eq. 1);
 *   - later timesteps: the LM input is sum_i gamma_i * E[last token of draft i] (Eq. 3) with
 *     gamma_i = p_i / sum_j p_j (Eq. 4); one LM pass over the shared context; the k most probable
 *     tokens are kept; draft i's n-gram distribution is sum_n lambda_n * p_n-gram (Eq. 5);
 *     p_f = p_theta^(1-alpha) * p_ngram^alpha (Eq. 6), or delta * p_theta^(1-alpha) when draft i's
 *     n-gram distribution shares no token with the kept ones (Eq. 7); the k*k options are ranked
 *     by p_i * p_f and the k best become the drafts (Eq. 2).
 * The LM is a Llama-style decoder (the paper names Llama-2 and does not restate it): pre-norm
 * residual blocks, RMSNorm, multi-head attention with rotary embedding on adjacent pairs,
 * SwiGLU feed-forward, final RMSNorm, untied output projection.
 *
 * Arithmetic: float64 throughout.  Quantisation points that belong to the model definition:
 * parameters are bf16; cached keys/values are rounded to float32 and then, if kv_dtype = 1, to
 * bf16 (round to nearest even); logits and candidate scores are rounded to float32 before any
 * ranking decision, with ties going to the lower index.
 *
 * Pins (tests/ without a GPU): logits against an independent dense float64 decoder written
 * with library matmuls; dense prefill against token-by-token decoding; k = 1 against a greedy
 * loop; the scoring stage against a brute-force enumeration of Eq. 5-7 in the linear domain with
 * dictionary counts; n-gram counts against a naive scan; closed forms for RMSNorm, rotary
 * embedding and single-position attention; the nucleus sampler against a brute-force search over all
 * token subsets, closed forms for uniform and two-point distributions, and draw frequencies.
 * Unpinned against the paper itself (it prints no
 * worked example): delta's value, where tau is applied, the per-draft reading of "no overlap",
 * and the absolute value of P.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_K 16
#define ORC_MAX_ORD 8

typedef struct {
  int32_t n_layers, d_model, n_heads, d_ffn, vocab, max_pos;
  double rms_eps, rope_theta;
  int32_t k, n_min, n_max;
  double lambda[ORC_MAX_ORD]; /* lambda[n - 2] */
  double alpha, tau, delta;
  int32_t kv_dtype;           /* 0: float32 cache, 1: bf16 cache */
  int32_t pad_;
} orc_config;

typedef struct {
  const uint16_t *tok_emb, *final_norm, *lm_head;
  const uint16_t *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
  const uint16_t *const *ffn_norm, *const *wgate, *const *wup, *const *wdown;
} orc_weights;

typedef struct {
  int32_t n;            /* order */
  int32_t pad_;
  int64_t n_entries;
  const int32_t *keys;  /* [n_entries][n], lexicographic */
  const int64_t *counts;
} orc_ngram;

typedef struct {
  orc_config c;
  orc_weights w;
  int n_tables;
  orc_ngram tab[ORC_MAX_ORD];
  float *kc, *vc;   /* [L][max_pos][d] cached keys / values (already quantised) */
  int32_t *draft;   /* [k][max_pos] full token sequences, prefix included */
  int32_t len;      /* tokens per draft */
  int32_t T;        /* cached positions */
  double logP[ORC_MAX_K], gamma[ORC_MAX_K];
  double *logits;   /* [vocab], last LM pass */
  double *trace;    /* [L][2][d]: last processed position's residual after attention / after FFN */
  const float *force_k, *force_v; /* [L][force_T][d] cache values to adopt where they are a valid rounding, or NULL */
  int force_T;
  double force_slack;
  int64_t force_flips, force_bad;
  double force_need;    /* largest slack an adopted value needed since the last orc_follow_cache */
  /* last step's intermediates */
  int32_t cand_tok[ORC_MAX_K];
  double cand_lp[ORC_MAX_K];
  double score[ORC_MAX_K * ORC_MAX_K];
  double png[ORC_MAX_K * ORC_MAX_K];
  int64_t cnt[ORC_MAX_K * ORC_MAX_K * ORC_MAX_ORD], tot[ORC_MAX_K * ORC_MAX_ORD];
  int32_t sel[ORC_MAX_K];
} orc_ctx;

/* ---------- scalar helpers ---------- */

static double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* float32 -> nearest bf16 (ties to even), returned as float32 */
float orc_round_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return f; /* NaN */
  u += 0x7fffu + ((u >> 16) & 1u);
  u &= 0xffff0000u;
  memcpy(&f, &u, 4);
  return f;
}

/* ---------- decoder pieces (each exported so the tests can pin it) ---------- */

/* y_j = x_j / sqrt(mean(x^2) + eps) * g_j */
void orc_rmsnorm(const double *x, const uint16_t *g, int d, double eps, double *y) {
  double ss = 0.0;
  for (int j = 0; j < d; ++j) ss += x[j] * x[j];
  double r = 1.0 / sqrt(ss / d + eps);
  for (int j = 0; j < d; ++j) y[j] = x[j] * r * bf16_to_double(g[j]);
}

/* rotary embedding of one head vector at position pos: pair (2i, 2i+1) turns by pos * theta^(-2i/hd) */
void orc_rope(double *x, int hd, int pos, double theta) {
  for (int i = 0; i < hd / 2; ++i) {
    double ang = (double)pos * pow(theta, -2.0 * i / hd);
    double c = cos(ang), s = sin(ang);
    double a = x[2 * i], b = x[2 * i + 1];
    x[2 * i] = a * c - b * s;
    x[2 * i + 1] = a * s + b * c;
  }
}

/* Y[t][r] = sum_c W[r][c] * X[t][c] for t < m */
static void matmul_rows(const uint16_t *W, int R, int C, const double *X, int m, double *Y) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < R; ++r) {
    const uint16_t *wr = W + (size_t)r * C;
    for (int t = 0; t < m; ++t) {
      const double *x = X + (size_t)t * C;
      double acc = 0.0;
      for (int c = 0; c < C; ++c) acc += bf16_to_double(wr[c]) * x[c];
      Y[(size_t)t * R + r] = acc;
    }
  }
}

/* softmax attention of one head's query over positions 0..T-1 of a cache with row stride d */
void orc_attention_head(const double *q, const float *K, const float *V, int T, int hd, int stride, double *o) {
  double *s = (double *)malloc(sizeof(double) * (size_t)T);
  double mx = -INFINITY;
  for (int t = 0; t < T; ++t) {
    double acc = 0.0;
    for (int j = 0; j < hd; ++j) acc += q[j] * (double)K[(size_t)t * stride + j];
    s[t] = acc / sqrt((double)hd);
    if (s[t] > mx) mx = s[t];
  }
  double den = 0.0;
  for (int t = 0; t < T; ++t) {
    s[t] = exp(s[t] - mx);
    den += s[t];
  }
  for (int j = 0; j < hd; ++j) {
    double acc = 0.0;
    for (int t = 0; t < T; ++t) acc += s[t] * (double)V[(size_t)t * stride + j];
    o[j] = acc / den;
  }
  free(s);
}

static float quant_kv(const orc_config *c, double x) {
  float f = (float)x;
  return c->kv_dtype == 1 ? orc_round_bf16(f) : f;
}

/*
 * The cache value for the exact value x.  Rounding to the cache type is a decision that float
 * rounding can tip either way when x lies within rounding error of the midpoint of two
 * representable values.  When the tests supply another implementation's cache value `other`, it is
 * adopted only if it is what round-to-nearest gives for some value within `slack` of x, i.e. if
 * round(x - slack) <= other <= round(x + slack) and `other` is representable (slack = the caller's
 * bound on the other side's float error in absolute terms).  With slack far below the local spacing
 * this admits the exact value's other neighbour only when x is within slack of the midpoint; a value
 * on the far side of the interval (x a tenth of the way from a to b, other = b), a truncation, or
 * anything further away is counted as a mismatch and not adopted.  Near zero, where the spacing is
 * below slack, it admits the few values a float error of that size can reach.  force_need keeps the
 * largest slack any adopted value needed, so that the tests can report how tight their bound is.
 */
static double kv_neighbour(const orc_config *c, float v, int upwards) {
  const uint32_t step = c->kv_dtype == 1 ? 0x10000u : 1u;
  uint32_t u;
  memcpy(&u, &v, 4);
  if (v == 0.0f) u = (upwards ? 0u : 0x80000000u) + step;
  else if ((v > 0.0f) == (upwards != 0)) u += step;   /* away from zero */
  else u -= step;                                     /* towards zero */
  float r;
  memcpy(&r, &u, 4);
  return (double)r;
}

static float follow_kv(orc_ctx *o, double x, const float *other) {
  float own = quant_kv(&o->c, x);
  if (!other) return own;
  if (*other == own) return own;
  const double v = (double)*other;
  const float lo = quant_kv(&o->c, x - o->force_slack), hi = quant_kv(&o->c, x + o->force_slack);
  if (quant_kv(&o->c, v) == *other && *other >= lo && *other <= hi) {
    /* the error that tips the rounding to `other`: distance from x to the nearer end of other's rounding interval */
    const double need = v > (double)own ? 0.5 * (v + kv_neighbour(&o->c, *other, 0)) - x
                                        : x - 0.5 * (v + kv_neighbour(&o->c, *other, 1));
    o->force_flips++;
    if (need > o->force_need) o->force_need = need;
    return *other;
  }
  o->force_bad++;
  return own;
}

/*
 * The decoder over m new positions pos0..pos0+m-1 whose input rows are X[m][d]; the positions
 * before pos0 are already in the cache.  Layer by layer over all new positions (the dense causal
 * pass); m = 1 is an ordinary cached decode step.  Leaves the final residual rows in X.
 */
static void decoder_forward(orc_ctx *o, double *X, int m, int pos0) {
  const orc_config *c = &o->c;
  const int d = c->d_model, f = c->d_ffn, H = c->n_heads, hd = d / H;
  double *A = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *Q = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *Kn = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *Vn = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *O = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *Y = (double *)malloc(sizeof(double) * (size_t)m * d);
  double *G = (double *)malloc(sizeof(double) * (size_t)m * f);
  double *U = (double *)malloc(sizeof(double) * (size_t)m * f);
  for (int l = 0; l < c->n_layers; ++l) {
    float *kc = o->kc + (size_t)l * c->max_pos * d;
    float *vc = o->vc + (size_t)l * c->max_pos * d;
    for (int t = 0; t < m; ++t) orc_rmsnorm(X + (size_t)t * d, o->w.attn_norm[l], d, c->rms_eps, A + (size_t)t * d);
    matmul_rows(o->w.wq[l], d, d, A, m, Q);
    matmul_rows(o->w.wk[l], d, d, A, m, Kn);
    matmul_rows(o->w.wv[l], d, d, A, m, Vn);
    for (int t = 0; t < m; ++t) {
      for (int h = 0; h < H; ++h) {
        orc_rope(Q + (size_t)t * d + h * hd, hd, pos0 + t, c->rope_theta);
        orc_rope(Kn + (size_t)t * d + h * hd, hd, pos0 + t, c->rope_theta);
      }
      for (int j = 0; j < d; ++j) {
        const int fp = pos0 + t;
        const float *fk = (o->force_k && fp < o->force_T) ? o->force_k + ((size_t)l * o->force_T + fp) * d + j : NULL;
        const float *fv = (o->force_v && fp < o->force_T) ? o->force_v + ((size_t)l * o->force_T + fp) * d + j : NULL;
        kc[(size_t)fp * d + j] = follow_kv(o, Kn[(size_t)t * d + j], fk);
        vc[(size_t)fp * d + j] = follow_kv(o, Vn[(size_t)t * d + j], fv);
      }
    }
#pragma omp parallel for collapse(2) schedule(static)
    for (int t = 0; t < m; ++t)
      for (int h = 0; h < H; ++h)
        orc_attention_head(Q + (size_t)t * d + h * hd, kc + h * hd, vc + h * hd, pos0 + t + 1, hd, d,
                           O + (size_t)t * d + h * hd);
    matmul_rows(o->w.wo[l], d, d, O, m, Y);
    for (size_t i = 0; i < (size_t)m * d; ++i) X[i] += Y[i];
    memcpy(o->trace + (size_t)(2 * l) * d, X + (size_t)(m - 1) * d, sizeof(double) * (size_t)d);
    for (int t = 0; t < m; ++t) orc_rmsnorm(X + (size_t)t * d, o->w.ffn_norm[l], d, c->rms_eps, A + (size_t)t * d);
    matmul_rows(o->w.wgate[l], f, d, A, m, G);
    matmul_rows(o->w.wup[l], f, d, A, m, U);
    for (size_t i = 0; i < (size_t)m * f; ++i) U[i] = G[i] / (1.0 + exp(-G[i])) * U[i];
    matmul_rows(o->w.wdown[l], d, f, U, m, Y);
    for (size_t i = 0; i < (size_t)m * d; ++i) X[i] += Y[i];
    memcpy(o->trace + (size_t)(2 * l + 1) * d, X + (size_t)(m - 1) * d, sizeof(double) * (size_t)d);
  }
  free(A); free(Q); free(Kn); free(Vn); free(O); free(Y); free(G); free(U);
}

/* logits of one residual row: W_head * RMSNorm(x) */
static void lm_head(orc_ctx *o, const double *x) {
  const orc_config *c = &o->c;
  double *a = (double *)malloc(sizeof(double) * (size_t)c->d_model);
  orc_rmsnorm(x, o->w.final_norm, c->d_model, c->rms_eps, a);
  matmul_rows(o->w.lm_head, c->vocab, c->d_model, a, 1, o->logits);
  free(a);
}

/*
 * KeepTopK (Algorithm 1) and the temperature: tok[j] = id of the j-th largest logit, ranking
 * float32-rounded logits, ties to the lower id; lp[j] = z/tau - log sum_v exp(z_v/tau) over the
 * whole vocabulary.
 */
void orc_topk_logprob(const double *z, int vocab, int k, double tau, int32_t *tok, double *lp) {
  for (int j = 0; j < k; ++j) {
    int best = -1;
    for (int v = 0; v < vocab; ++v) {
      int taken = 0;
      for (int i = 0; i < j; ++i) taken |= (tok[i] == v);
      if (taken) continue;
      if (best < 0 || (float)z[v] > (float)z[best]) best = v;
    }
    tok[j] = best;
  }
  double mx = -INFINITY;
  for (int v = 0; v < vocab; ++v)
    if (z[v] / tau > mx) mx = z[v] / tau;
  double den = 0.0;
  for (int v = 0; v < vocab; ++v) den += exp(z[v] / tau - mx);
  double lse = mx + log(den);
  for (int j = 0; j < k; ++j) lp[j] = z[tok[j]] / tau - lse;
}

/*
 * Nucleus sampling (Section 2: the smallest set of tokens whose cumulative probability reaches p, then a
 * draw from that set in proportion to probability; Section 4.5 uses such generations as prefixes for SPD).
 * prob = softmax(z / temperature); tokens are taken by descending probability, equal ones by ascending id;
 * the nucleus is the shortest head of that order whose cumulative probability is >= p; with the uniform
 * number u in [0, 1) the drawn token is the first whose cumulative probability exceeds u * (mass of the
 * nucleus).  Returns the token.  info (may be NULL) receives: [0] size of the nucleus, [1] its mass,
 * [2] distance from p to the nearest cumulative probability next to the cut, [3] distance from u * mass to
 * the nearer end of the drawn token's interval.
 */
typedef struct { double z; int32_t id; } ns_item;
static int ns_cmp(const void *a, const void *b) {
  const ns_item *x = (const ns_item *)a, *y = (const ns_item *)b;
  if (x->z > y->z) return -1;
  if (x->z < y->z) return 1;
  return x->id < y->id ? -1 : (x->id > y->id ? 1 : 0);
}
int32_t orc_nucleus(const double *z, int vocab, double temperature, double p, double u, double *info) {
  ns_item *it = (ns_item *)malloc(sizeof(ns_item) * (size_t)vocab);
  double mx = -INFINITY, den = 0.0;
  for (int v = 0; v < vocab; ++v)
    if (z[v] / temperature > mx) mx = z[v] / temperature;
  for (int v = 0; v < vocab; ++v) den += exp(z[v] / temperature - mx);
  for (int v = 0; v < vocab; ++v) {
    it[v].z = z[v];
    it[v].id = v;
  }
  qsort(it, (size_t)vocab, sizeof(ns_item), ns_cmp);
  /* the cut */
  double cum = 0.0, before = 0.0;
  int size = 0;
  while (size < vocab) {
    before = cum;
    cum += exp(it[size].z / temperature - mx) / den;
    ++size;
    if (cum >= p) break;
  }
  const double mass = cum;
  const double gap_cut = fmin(fabs(cum - p), fabs(p - before));
  /* the draw */
  const double target = u * mass;
  double run = 0.0, lo = 0.0;
  int pick = size - 1;
  for (int i = 0; i < size; ++i) {
    lo = run;
    run += exp(it[i].z / temperature - mx) / den;
    if (run > target) {
      pick = i;
      break;
    }
  }
  if (info) {
    info[0] = (double)size;
    info[1] = mass;
    info[2] = gap_cut;
    info[3] = fmin(target - lo, run - target);
  }
  const int32_t tok = it[pick].id;
  free(it);
  return tok;
}

/* gamma_i = p_i / sum_j p_j with p = exp(logP)  (Eq. 4) */
void orc_gamma(const double *logP, int k, double *gamma) {
  double mx = -INFINITY, den = 0.0;
  for (int i = 0; i < k; ++i)
    if (logP[i] > mx) mx = logP[i];
  for (int i = 0; i < k; ++i) den += exp(logP[i] - mx);
  for (int i = 0; i < k; ++i) gamma[i] = exp(logP[i] - mx) / den;
}

/* ---------- n-gram store: sorted unique n-grams with counts ---------- */

static int cmp_prefix(const int32_t *row, const int32_t *key, int len) {
  for (int j = 0; j < len; ++j) {
    if (row[j] < key[j]) return -1;
    if (row[j] > key[j]) return 1;
  }
  return 0;
}

/* first row whose first `len` tokens are >= key (strict = 0) or > key (strict = 1) */
static int64_t bound(const orc_ngram *t, const int32_t *key, int len, int strict) {
  int64_t lo = 0, hi = t->n_entries;
  while (lo < hi) {
    int64_t mid = lo + (hi - lo) / 2;
    int c = cmp_prefix(t->keys + (size_t)mid * t->n, key, len);
    if (c < 0 || (strict && c == 0)) lo = mid + 1; else hi = mid;
  }
  return lo;
}

/*
 * Counts behind p_n(tok | ctx) for one table: *tot = sum of the counts of every stored n-gram
 * that starts with the n-1 context tokens, *cnt = count of ctx followed by tok (0 if absent).
 */
void orc_ngram_counts(const orc_ngram *t, const int32_t *ctx, int32_t tok, int64_t *cnt, int64_t *tot) {
  int32_t key[ORC_MAX_ORD];
  for (int j = 0; j < t->n - 1; ++j) key[j] = ctx[j];
  key[t->n - 1] = tok;
  int64_t a = bound(t, key, t->n - 1, 0), b = bound(t, key, t->n - 1, 1);
  int64_t s = 0;
  for (int64_t i = a; i < b; ++i) s += t->counts[i];
  *tot = s;
  int64_t e = bound(t, key, t->n, 0);
  *cnt = (e < t->n_entries && cmp_prefix(t->keys + (size_t)e * t->n, key, t->n) == 0) ? t->counts[e] : 0;
}

/*
 * Eq. 5 for one (draft history, token): sum over stored orders n of lambda_n * count(ctx, tok) /
 * total(ctx), ctx = the last n-1 tokens of the history (prefix tokens included).  An order whose
 * context is longer than the history, or unseen, contributes 0.  cnt/tot (one entry per table, in
 * table order) receive the integers used; -1 marks a skipped order.
 */
double orc_png(const orc_config *c, const orc_ngram *tabs, int n_tables, const int32_t *hist, int hist_len,
               int32_t tok, int64_t *cnt, int64_t *tot) {
  double p = 0.0;
  for (int ti = 0; ti < n_tables; ++ti) {
    const orc_ngram *t = &tabs[ti];
    cnt[ti] = tot[ti] = -1;
    if (t->n < c->n_min || t->n > c->n_max || hist_len < t->n - 1) continue;
    orc_ngram_counts(t, hist + hist_len - (t->n - 1), tok, &cnt[ti], &tot[ti]);
    if (tot[ti] > 0) p += c->lambda[t->n - 2] * ((double)cnt[ti] / (double)tot[ti]);
  }
  return p;
}

/*
 * Scoring stage of one timestep (Eq. 2, 5, 6, 7 in the log domain).  For draft i (history
 * hist + i*hist_stride, hist_len tokens, log-probability logP[i]) and kept token j (cand_tok[j],
 * log-probability cand_lp[j]):
 *   score(i,j) = logP[i] + (1-alpha)*cand_lp[j] + alpha*log(png(i,j))   if draft i's n-gram
 *                distribution gives at least one kept token a non-zero probability and png(i,j) > 0,
 *              = -inf                                                    if it does and png(i,j) = 0,
 *              = logP[i] + (1-alpha)*cand_lp[j] + log(delta)             if it gives none (Eq. 7).
 * The k largest float32-rounded scores win (ties to the lower i*k + j); sel[] lists them in
 * descending order, new_logP their scores and new_gamma Eq. 4 of those.
 */
void orc_score_stage(const orc_config *c, const orc_ngram *tabs, int n_tables, const int32_t *hist, int hist_stride,
                     int hist_len, const double *logP, const int32_t *cand_tok, const double *cand_lp,
                     double *png, double *score, int64_t *cnt, int64_t *tot, int32_t *sel, double *new_logP,
                     double *new_gamma) {
  const int k = c->k;
  for (int i = 0; i < k; ++i) {
    int overlap = 0;
    for (int j = 0; j < k; ++j) {
      int64_t tt[ORC_MAX_ORD];
      png[i * k + j] = orc_png(c, tabs, n_tables, hist + (size_t)i * hist_stride, hist_len, cand_tok[j],
                               cnt + (size_t)(i * k + j) * ORC_MAX_ORD, tt);
      for (int ti = 0; ti < n_tables; ++ti) tot[i * ORC_MAX_ORD + ti] = tt[ti];
      if (png[i * k + j] > 0.0) overlap = 1;
    }
    for (int j = 0; j < k; ++j) {
      double base = logP[i] + (1.0 - c->alpha) * cand_lp[j];
      if (!overlap) score[i * k + j] = base + log(c->delta);
      else if (png[i * k + j] > 0.0) score[i * k + j] = base + c->alpha * log(png[i * k + j]);
      else score[i * k + j] = -INFINITY;
    }
  }
  for (int r = 0; r < k; ++r) {
    int best = -1;
    for (int q = 0; q < k * k; ++q) {
      int taken = 0;
      for (int i = 0; i < r; ++i) taken |= (sel[i] == q);
      if (taken) continue;
      if (best < 0 || (float)score[q] > (float)score[best]) best = q;
    }
    sel[r] = best;
    new_logP[r] = score[best];
  }
  orc_gamma(new_logP, k, new_gamma);
}

/* ---------- the procedure ---------- */

orc_ctx *orc_create(const orc_config *c, const orc_weights *w, const orc_ngram *tabs, int n_tables) {
  if (c->k < 1 || c->k > ORC_MAX_K || n_tables > ORC_MAX_ORD || c->d_model % c->n_heads) return NULL;
  orc_ctx *o = (orc_ctx *)calloc(1, sizeof(orc_ctx));
  o->c = *c;
  o->w = *w;
  o->n_tables = n_tables;
  for (int i = 0; i < n_tables; ++i) o->tab[i] = tabs[i];
  size_t kv = (size_t)c->n_layers * c->max_pos * c->d_model;
  o->kc = (float *)calloc(kv, sizeof(float));
  o->vc = (float *)calloc(kv, sizeof(float));
  o->draft = (int32_t *)calloc((size_t)c->k * c->max_pos, sizeof(int32_t));
  o->logits = (double *)calloc((size_t)c->vocab, sizeof(double));
  o->trace = (double *)calloc((size_t)c->n_layers * 2 * c->d_model, sizeof(double));
  return o;
}

void orc_destroy(orc_ctx *o) {
  if (!o) return;
  free(o->kc); free(o->vc); free(o->draft); free(o->logits); free(o->trace); free(o);
}

static void embed_row(const orc_ctx *o, int32_t tok, double *x) {
  const uint16_t *e = o->w.tok_emb + (size_t)tok * o->c.d_model;
  for (int j = 0; j < o->c.d_model; ++j) x[j] = bf16_to_double(e[j]);
}

/*
 * First timestep (Eq. 1): dense pass over the prefix, drafts = prefix + i-th most probable token,
 * logP_i = its log-probability, no n-gram term.  Returns 0, or -1 on bad arguments.
 */
int orc_prefill(orc_ctx *o, const int32_t *ids, int m, int32_t *out_ids, double *out_gamma) {
  const orc_config *c = &o->c;
  if (m < 1 || m >= c->max_pos) return -1;
  for (int t = 0; t < m; ++t)
    if (ids[t] < 0 || ids[t] >= c->vocab) return -1;
  double *X = (double *)malloc(sizeof(double) * (size_t)m * c->d_model);
  for (int t = 0; t < m; ++t) embed_row(o, ids[t], X + (size_t)t * c->d_model);
  decoder_forward(o, X, m, 0);
  lm_head(o, X + (size_t)(m - 1) * c->d_model);
  free(X);
  o->T = m;
  orc_topk_logprob(o->logits, c->vocab, c->k, c->tau, o->cand_tok, o->cand_lp);
  for (int i = 0; i < c->k; ++i) {
    int32_t *dr = o->draft + (size_t)i * c->max_pos;
    for (int t = 0; t < m; ++t) dr[t] = ids[t];
    dr[m] = o->cand_tok[i];
    o->logP[i] = o->cand_lp[i];
    o->sel[i] = i;
  }
  o->len = m + 1;
  orc_gamma(o->logP, c->k, o->gamma);
  for (int i = 0; i < c->k; ++i) {
    out_ids[i] = o->cand_tok[i];
    out_gamma[i] = o->gamma[i];
  }
  return 0;
}

/*
 * Ordinary cached decoding of one plain token at the next position (no drafts involved); fills
 * the logits.  Used to check that the dense pass and token-by-token decoding agree.
 */
int orc_feed_token(orc_ctx *o, int32_t tok) {
  const orc_config *c = &o->c;
  if (tok < 0 || tok >= c->vocab || o->T + 1 > c->max_pos) return -1;
  double *x = (double *)malloc(sizeof(double) * (size_t)c->d_model);
  embed_row(o, tok, x);
  decoder_forward(o, x, 1, o->T);
  lm_head(o, x);
  free(x);
  o->T += 1;
  return 0;
}

/* Eq. 3 + one LM pass on the superposed input at the next position; fills logits and candidates. */
int orc_step_forward(orc_ctx *o) {
  const orc_config *c = &o->c;
  if (o->len < 1 || o->T + 1 > c->max_pos || o->len + 1 > c->max_pos) return -1;
  double *x = (double *)calloc((size_t)c->d_model, sizeof(double));
  double *e = (double *)malloc(sizeof(double) * (size_t)c->d_model);
  for (int i = 0; i < c->k; ++i) {
    embed_row(o, o->draft[(size_t)i * c->max_pos + o->len - 1], e);
    for (int j = 0; j < c->d_model; ++j) x[j] += o->gamma[i] * e[j];
  }
  decoder_forward(o, x, 1, o->T);
  lm_head(o, x);
  free(x); free(e);
  o->T += 1;
  orc_topk_logprob(o->logits, c->vocab, c->k, c->tau, o->cand_tok, o->cand_lp);
  return 0;
}

/* Scores the k*k options of the current candidates against the current drafts; fills sel. */
void orc_step_score(orc_ctx *o, double *new_logP, double *new_gamma) {
  orc_score_stage(&o->c, o->tab, o->n_tables, o->draft, o->c.max_pos, o->len, o->logP, o->cand_tok, o->cand_lp,
                  o->png, o->score, o->cnt, o->tot, o->sel, new_logP, new_gamma);
}

/*
 * Makes option sel[r] = i*k + j the new draft r: draft i's tokens followed by candidate j, with
 * log-probability new_logP[r].  (The tests use it to let the oracle follow another
 * implementation's choice on steps where two options tie within rounding.)
 */
void orc_step_commit(orc_ctx *o, const int32_t *sel, const double *new_logP) {
  const orc_config *c = &o->c;
  const int k = c->k;
  int32_t *nd = (int32_t *)malloc(sizeof(int32_t) * (size_t)k * c->max_pos);
  for (int r = 0; r < k; ++r) {
    int i = sel[r] / k, j = sel[r] % k;
    memcpy(nd + (size_t)r * c->max_pos, o->draft + (size_t)i * c->max_pos, sizeof(int32_t) * (size_t)o->len);
    nd[(size_t)r * c->max_pos + o->len] = o->cand_tok[j];
    o->logP[r] = new_logP[r];
    o->sel[r] = sel[r];
  }
  memcpy(o->draft, nd, sizeof(int32_t) * (size_t)k * c->max_pos);
  free(nd);
  o->len += 1;
  orc_gamma(o->logP, k, o->gamma);
}

/*
 * Gives the next LM passes another implementation's cache contents ([L][T][d] keys and values as float32)
 * to follow wherever they are a valid rounding of this oracle's exact values (to within `slack`, see
 * follow_kv); NULL switches it off.
 * flips / bad (either may be NULL) report how many values were adopted / refused since the last call.
 */
double orc_follow_need(const orc_ctx *o) { return o->force_need; }

void orc_follow_cache(orc_ctx *o, const float *k, const float *v, int T, double slack, int64_t *flips, int64_t *bad) {
  if (flips) *flips = o->force_flips;
  if (bad) *bad = o->force_bad;
  o->force_k = k;
  o->force_v = v;
  o->force_T = T;
  o->force_slack = slack;
  o->force_flips = o->force_bad = 0;
  o->force_need = 0.0;
}

/*
 * Replaces the draft log-probabilities (and with them gamma, Eq. 4).  The tests use it so that a
 * stage-by-stage comparison feeds both implementations the same superposed input: at tau = 0.06 a logit
 * difference of e moves a log-probability by e / tau, so rounding-level differences in one step's logits
 * would otherwise change the next step's input.
 */
void orc_set_logP(orc_ctx *o, const double *logP) {
  for (int i = 0; i < o->c.k; ++i) o->logP[i] = logP[i];
  orc_gamma(o->logP, o->c.k, o->gamma);
}

/* One later timestep of Algorithm 1.  out_parent[r] = index of the draft that new draft r extends. */
int orc_step(orc_ctx *o, int32_t *out_ids, int32_t *out_parent, double *out_gamma) {
  double nl[ORC_MAX_K], ng[ORC_MAX_K];
  int32_t sel[ORC_MAX_K];
  if (orc_step_forward(o)) return -1;
  orc_step_score(o, nl, ng);
  for (int r = 0; r < o->c.k; ++r) sel[r] = o->sel[r];
  orc_step_commit(o, sel, nl);
  for (int r = 0; r < o->c.k; ++r) {
    out_ids[r] = o->cand_tok[sel[r] % o->c.k];
    out_parent[r] = sel[r] / o->c.k;
    out_gamma[r] = o->gamma[r];
  }
  return 0;
}

/* ---------- read-outs for the tests ---------- */

const double *orc_logits(const orc_ctx *o) { return o->logits; }
const double *orc_trace(const orc_ctx *o) { return o->trace; }
const double *orc_logP(const orc_ctx *o) { return o->logP; }
const double *orc_gamma_now(const orc_ctx *o) { return o->gamma; }
const int32_t *orc_cand_tok(const orc_ctx *o) { return o->cand_tok; }
const double *orc_cand_lp(const orc_ctx *o) { return o->cand_lp; }
const double *orc_scores(const orc_ctx *o) { return o->score; }
const double *orc_png_last(const orc_ctx *o) { return o->png; }
const int64_t *orc_cnt_last(const orc_ctx *o) { return o->cnt; }
const int64_t *orc_tot_last(const orc_ctx *o) { return o->tot; }
const int32_t *orc_sel_last(const orc_ctx *o) { return o->sel; }
const int32_t *orc_drafts(const orc_ctx *o) { return o->draft; }
int orc_len(const orc_ctx *o) { return o->len; }
int orc_T(const orc_ctx *o) { return o->T; }
const float *orc_kcache(const orc_ctx *o) { return o->kc; }
const float *orc_vcache(const orc_ctx *o) { return o->vc; }
int orc_max_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
