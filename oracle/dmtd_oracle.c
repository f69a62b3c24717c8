/*
 * CPU oracle for the DMTD decode path.  TEST INFRASTRUCTURE, NOT PRODUCT: see dmtd_oracle.h.
 *
 * Everything here is written for reading, not speed: one loop nest per formula, doubles
 * throughout, no blocking, no fusion.  OpenMP is used only to run independent output
 * elements on different cores; it never changes the order of a summation.
 */
#include "dmtd_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ storage widening */

static double load_weight(const void *W, int dtype, size_t i) {
  if (dtype == ORACLE_BF16) {
    /* a bf16 value is the top 16 bits of an IEEE fp32 */
    uint32_t bits = (uint32_t)((const uint16_t *)W)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
  return (double)((const float *)W)[i];
}

static void widen_row(const void *W, int dtype, size_t row, int n, double *dst) {
  for (int i = 0; i < n; ++i) dst[i] = load_weight(W, dtype, row * (size_t)n + (size_t)i);
}

/* ------------------------------------------------------------------ unit functions */

void oracle_rmsnorm(const double *x, const double *w, double eps, int rows, int n, double *y) {
  for (int r = 0; r < rows; ++r) {
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[(size_t)r * n + i] * x[(size_t)r * n + i];
    double inv = 1.0 / sqrt(ss / (double)n + eps);
    for (int i = 0; i < n; ++i) y[(size_t)r * n + i] = x[(size_t)r * n + i] * inv * w[i];
  }
}

void oracle_rope(double *v, int head_dim, int pos, double theta) {
  int half = head_dim / 2;
  for (int i = 0; i < half; ++i) {
    double freq = pow(theta, -2.0 * (double)i / (double)head_dim);
    double ang = (double)pos * freq;
    double c = cos(ang), s = sin(ang);
    double a = v[i], b = v[i + half];
    v[i] = a * c - b * s;
    v[i + half] = b * c + a * s;
  }
}

void oracle_attention(const double *q, const double *k, const double *v, int R, int pos0,
                      int nq, int nkv, int d, double *out) {
  int group = nq / nkv;                  /* query heads per KV head */
  double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(static)
  for (int r = 0; r < R; ++r) {
    for (int h = 0; h < nq; ++h) {
      int n_keys = pos0 + r + 1;         /* causal: keys 0 .. own position */
      int kvh = h / group;
      const double *qv = q + ((size_t)r * nq + h) * d;
      double *score = (double *)malloc((size_t)n_keys * sizeof(double));
      double top = -INFINITY;
      for (int j = 0; j < n_keys; ++j) {
        const double *kj = k + ((size_t)j * nkv + kvh) * d;
        double dot = 0.0;
        for (int i = 0; i < d; ++i) dot += qv[i] * kj[i];
        score[j] = dot * scale;
        if (score[j] > top) top = score[j];
      }
      double denom = 0.0;
      for (int j = 0; j < n_keys; ++j) {
        score[j] = exp(score[j] - top);
        denom += score[j];
      }
      double *o = out + ((size_t)r * nq + h) * d;
      for (int i = 0; i < d; ++i) o[i] = 0.0;
      for (int j = 0; j < n_keys; ++j) {
        const double *vj = v + ((size_t)j * nkv + kvh) * d;
        double wj = score[j] / denom;
        for (int i = 0; i < d; ++i) o[i] += wj * vj[i];
      }
      free(score);
    }
  }
}

void oracle_linear(const void *W, int dtype, int n_out, int n_in, const double *x, int rows,
                   double *y) {
#pragma omp parallel
  {
    double *wrow = (double *)malloc((size_t)n_in * sizeof(double));
#pragma omp for schedule(static)
    for (int o = 0; o < n_out; ++o) {
      widen_row(W, dtype, (size_t)o, n_in, wrow);
      for (int r = 0; r < rows; ++r) {
        const double *xr = x + (size_t)r * n_in;
        double acc = 0.0;
        /* the simd clause lets the compiler keep several partial sums; the sum is the same
         * up to rounding order */
#pragma omp simd reduction(+ : acc)
        for (int k = 0; k < n_in; ++k) acc += wrow[k] * xr[k];
        y[(size_t)r * n_out + o] = acc;
      }
    }
    free(wrow);
  }
}

double oracle_silu(double t) { return t / (1.0 + exp(-t)); }

double oracle_plt(int L, int L_d, int tau) {
  return ((double)L + (double)(tau - 1) * (double)L_d) / ((double)tau * (double)L);
}

/* ------------------------------------------------------------------ model pieces */

static double *widen_vector(const void *w, int dtype, int n) {
  double *v = (double *)malloc((size_t)n * sizeof(double));
  for (int i = 0; i < n; ++i) v[i] = load_weight(w, dtype, (size_t)i);
  return v;
}

static void embed_rows(const oracle_shape *s, const oracle_weights *w, const int32_t *tok,
                       int rows, double *x) {
  for (int r = 0; r < rows; ++r)
    widen_row(w->embed, s->weight_dtype, (size_t)tok[r], s->hidden, x + (size_t)r * s->hidden);
}

/* One decoder layer on R rows of one sequence at positions pos0..pos0+R-1.
 * kc, vc: that layer's and that sequence's cache, [max_seq][nkv][d].  x [R][hidden] in/out. */
static void layer_forward(const oracle_shape *s, const oracle_layer_weights *lw, double *x,
                          int R, int pos0, double *kc, double *vc) {
  int H = s->hidden, nq = s->n_q_heads, nkv = s->n_kv_heads, d = s->head_dim;
  int I = s->intermediate, dt = s->weight_dtype;
  int qd = nq * d, kvd = nkv * d;
  double *w_in = widen_vector(lw->input_norm, dt, H);
  double *w_post = widen_vector(lw->post_norm, dt, H);
  double *w_qn = widen_vector(lw->q_norm, dt, d);
  double *w_kn = widen_vector(lw->k_norm, dt, d);
  double *a = (double *)malloc((size_t)R * H * sizeof(double));
  double *q = (double *)malloc((size_t)R * qd * sizeof(double));
  double *k = (double *)malloc((size_t)R * kvd * sizeof(double));
  double *v = (double *)malloc((size_t)R * kvd * sizeof(double));
  double *o = (double *)malloc((size_t)R * qd * sizeof(double));
  double *t = (double *)malloc((size_t)R * H * sizeof(double));
  double *g = (double *)malloc((size_t)R * I * sizeof(double));
  double *u = (double *)malloc((size_t)R * I * sizeof(double));

  /* attention block */
  oracle_rmsnorm(x, w_in, s->rms_eps, R, H, a);
  oracle_linear(lw->q_proj, dt, qd, H, a, R, q);
  oracle_linear(lw->k_proj, dt, kvd, H, a, R, k);
  oracle_linear(lw->v_proj, dt, kvd, H, a, R, v);
  for (int r = 0; r < R; ++r) {
    int pos = pos0 + r;
    for (int h = 0; h < nq; ++h) {
      double *qh = q + ((size_t)r * nq + h) * d;
      oracle_rmsnorm(qh, w_qn, s->rms_eps, 1, d, qh);
      oracle_rope(qh, d, pos, s->rope_theta);
    }
    for (int h = 0; h < nkv; ++h) {
      double *kh = k + ((size_t)r * nkv + h) * d;
      oracle_rmsnorm(kh, w_kn, s->rms_eps, 1, d, kh);
      oracle_rope(kh, d, pos, s->rope_theta);
    }
    memcpy(kc + (size_t)pos * kvd, k + (size_t)r * kvd, (size_t)kvd * sizeof(double));
    memcpy(vc + (size_t)pos * kvd, v + (size_t)r * kvd, (size_t)kvd * sizeof(double));
  }
  oracle_attention(q, kc, vc, R, pos0, nq, nkv, d, o);
  oracle_linear(lw->o_proj, dt, H, qd, o, R, t);
  for (size_t i = 0; i < (size_t)R * H; ++i) x[i] += t[i];

  /* MLP block */
  oracle_rmsnorm(x, w_post, s->rms_eps, R, H, a);
  oracle_linear(lw->gate_proj, dt, I, H, a, R, g);
  oracle_linear(lw->up_proj, dt, I, H, a, R, u);
  for (size_t i = 0; i < (size_t)R * I; ++i) g[i] = oracle_silu(g[i]) * u[i];
  oracle_linear(lw->down_proj, dt, H, I, g, R, t);
  for (size_t i = 0; i < (size_t)R * H; ++i) x[i] += t[i];

  free(w_in); free(w_post); free(w_qn); free(w_kn);
  free(a); free(q); free(k); free(v); free(o); free(t); free(g); free(u);
}

/* logits [rows][vocab] = rmsnorm(x) * final_norm, times the embedding matrix transposed */
static void lm_head(const oracle_shape *s, const oracle_weights *w, const double *x, int rows,
                    double *logits) {
  double *wf = widen_vector(w->final_norm, s->weight_dtype, s->hidden);
  double *a = (double *)malloc((size_t)rows * s->hidden * sizeof(double));
  oracle_rmsnorm(x, wf, s->rms_eps, rows, s->hidden, a);
  oracle_linear(w->embed, s->weight_dtype, s->vocab, s->hidden, a, rows, logits);
  free(wf); free(a);
}

static int32_t argmax_lowest(const double *z, int n) {
  int32_t best = 0;
  for (int i = 1; i < n; ++i)
    if (z[i] > z[best]) best = i;      /* strict: the lowest index wins a tie */
  return best;
}

/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
 * SC'11): a counter-based generator - the four output words are a fixed function of a 128-bit
 * counter and a 64-bit key, so the CUDA path can draw the same numbers with no shared state. */
void oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Sampling from softmax(z / T) by the Gumbel-max rule: argmax_i (z_i / T + g_i) with independent
 * standard Gumbel noise g_i = -log(-log(u_i)).  u_i in (0, 1) comes from the top 24 bits of word i mod 4 of
 * Philox(counter = (i / 4, position, sequence, 0), key = seed): the draw depends only on the
 * seed, the position the token will take, the sequence index and the vocabulary index.  The
 * lowest index wins a tie, as in the greedy rule (T <= 0 means greedy). */
int32_t oracle_sample_token(const double *z, int n, double temperature, uint64_t seed, int32_t position,
                            int32_t sequence) {
  if (!(temperature > 0.0)) return argmax_lowest(z, n);
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  int32_t best = 0;
  double best_v = -INFINITY;
  for (int i = 0; i < n; ++i) {
    uint32_t ctr[4] = {(uint32_t)(i >> 2), (uint32_t)position, (uint32_t)sequence, 0u}, r[4];
    oracle_philox4x32(ctr, key, r);
    double u = ((double)(r[i & 3] >> 8) + 0.5) * (1.0 / 16777216.0);      /* the word's top 24 bits: exact in fp32 too */
    double v = z[i] / temperature - log(-log(u));
    if (v > best_v) { best_v = v; best = i; }
  }
  return best;
}

static int shape_ok(const oracle_shape *s) {
  if (!s) return 0;
  if (s->n_layers < 1 || s->hidden < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1) return 0;
  if (s->head_dim < 2 || (s->head_dim & 1) || s->intermediate < 1 || s->vocab < 1) return 0;
  if (s->n_q_heads % s->n_kv_heads) return 0;
  if (s->weight_dtype != ORACLE_F32 && s->weight_dtype != ORACLE_BF16) return 0;
  return 1;
}

/* ------------------------------------------------------------------ DMTD context */

struct oracle_ctx {
  oracle_shape s;
  oracle_weights w;
  oracle_layer_weights *layers;
  int32_t L_d, tau, max_batch, max_seq, B, literal_sum;
  double temperature;     /* > 0: sample by the Gumbel-max rule; 0: greedy */
  uint64_t sample_seed;
  int32_t L_e;            /* encoding layers reused by the short passes (the ExDy variant); 0 = none */
  double *h_enc;          /* [max_batch][max_seq][hidden]: output of the encoding layers at every decode position */
  double *kc, *vc;        /* [n_layers][max_batch][max_seq][nkv*d] */
  int32_t *tokens;        /* [max_batch][max_seq] */
  oracle_state st;
  int prefilled;
  oracle_pass_record *trace;
  int32_t n_trace, cap_trace;
  int64_t *calls, *rows;
};

static size_t cache_stride_seq(const oracle_ctx *c) {
  return (size_t)c->max_seq * c->s.n_kv_heads * c->s.head_dim;
}
double *oracle_k_cache(oracle_ctx *c, int32_t layer, int32_t b) {
  return c->kc + ((size_t)layer * c->max_batch + b) * cache_stride_seq(c);
}
double *oracle_v_cache(oracle_ctx *c, int32_t layer, int32_t b) {
  return c->vc + ((size_t)layer * c->max_batch + b) * cache_stride_seq(c);
}

int oracle_create(const oracle_shape *shape, int32_t L_d, int32_t tau, int32_t max_batch,
                  int32_t max_seq, const oracle_weights *w, oracle_ctx **out) {
  if (!shape_ok(shape) || !w || !out) return -1;
  if (L_d < 1 || L_d > shape->n_layers || tau < 1 || max_batch < 1 || max_seq < 1) return -2;
  oracle_ctx *c = (oracle_ctx *)calloc(1, sizeof *c);
  c->s = *shape;
  c->w = *w;
  c->layers = (oracle_layer_weights *)malloc((size_t)shape->n_layers * sizeof *c->layers);
  memcpy(c->layers, w->layers, (size_t)shape->n_layers * sizeof *c->layers);
  c->w.layers = c->layers;
  c->L_d = L_d; c->tau = tau; c->max_batch = max_batch; c->max_seq = max_seq;
  size_t n = (size_t)shape->n_layers * max_batch * cache_stride_seq(c);
  c->kc = (double *)calloc(n, sizeof(double));
  c->vc = (double *)calloc(n, sizeof(double));
  c->tokens = (int32_t *)calloc((size_t)max_batch * max_seq, sizeof(int32_t));
  c->h_enc = (double *)calloc((size_t)max_batch * max_seq * shape->hidden, sizeof(double));
  c->calls = (int64_t *)calloc((size_t)shape->n_layers, sizeof(int64_t));
  c->rows = (int64_t *)calloc((size_t)shape->n_layers, sizeof(int64_t));
  if (!c->kc || !c->vc || !c->tokens || !c->h_enc) { oracle_destroy(c); return -4; }
  oracle_reset(c);
  *out = c;
  return 0;
}

void oracle_destroy(oracle_ctx *c) {
  if (!c) return;
  free(c->layers); free(c->kc); free(c->vc); free(c->tokens); free(c->trace); free(c->h_enc);
  free(c->calls); free(c->rows); free(c);
}

int oracle_reset(oracle_ctx *c) {
  if (!c) return -1;
  memset(&c->st, 0, sizeof c->st);
  c->st.tau = c->tau; c->st.L_d = c->L_d;
  c->prefilled = 0; c->B = 0; c->n_trace = 0;
  memset(c->calls, 0, (size_t)c->s.n_layers * sizeof(int64_t));
  memset(c->rows, 0, (size_t)c->s.n_layers * sizeof(int64_t));
  return 0;
}

int oracle_set_tau(oracle_ctx *c, int32_t tau) {
  if (!c || tau < 1) return -1;
  if (c->prefilled && c->st.slot != 0) return -3;    /* only at a cycle boundary */
  c->tau = tau; c->st.tau = tau;
  return 0;
}

int oracle_set_encoding_layers(oracle_ctx *c, int32_t L_e) {
  if (!c || L_e < 0) return -1;
  if (c->prefilled) return -3;                          /* a property of the whole generation */
  if (L_e + c->L_d > c->s.n_layers) return -2;
  c->L_e = L_e;
  return 0;
}

int oracle_set_sampling(oracle_ctx *c, double temperature, uint64_t seed) {
  if (!c || !(temperature >= 0.0)) return -1;
  c->temperature = temperature;
  c->sample_seed = seed;
  return 0;
}

int oracle_set_literal_sum(oracle_ctx *c, int32_t on) {
  if (!c) return -1;
  c->literal_sum = on ? 1 : 0;
  return 0;
}

static void record_pass(oracle_ctx *c, int kind, int lb, int le, int ub, int ue) {
  if (c->n_trace == c->cap_trace) {
    c->cap_trace = c->cap_trace ? 2 * c->cap_trace : 64;
    c->trace = (oracle_pass_record *)realloc(c->trace, (size_t)c->cap_trace * sizeof *c->trace);
  }
  oracle_pass_record r = {kind, lb, le, ub, ue, c->st.cycle};
  c->trace[c->n_trace++] = r;
}

/* Layers [l0, l1) for every sequence of the batch; x [B][R][hidden]. */
static void run_layers(oracle_ctx *c, int l0, int l1, double *x, int B, int R, int pos0) {
  for (int l = l0; l < l1; ++l) {
    for (int b = 0; b < B; ++b)
      layer_forward(&c->s, &c->layers[l], x + (size_t)b * R * c->s.hidden, R, pos0,
                    oracle_k_cache(c, l, b), oracle_v_cache(c, l, b));
    c->calls[l] += 1;
    c->rows[l] += R;
  }
}

/* Head on one row per sequence, pick / force the next token, append it at n_known. */
static void emit(oracle_ctx *c, const double *x_last /*[B][hidden]*/, const int32_t *forced,
                 int forced_stride, int32_t *out_token, int out_stride, double *out_logits) {
  int B = c->B, V = c->s.vocab;
  double *z = (double *)malloc((size_t)B * V * sizeof(double));
  lm_head(&c->s, &c->w, x_last, B, z);
  for (int b = 0; b < B; ++b) {
    int32_t pick = oracle_sample_token(z + (size_t)b * V, V, c->temperature, c->sample_seed, c->st.n_known, b);
    if (out_token) out_token[(size_t)b * out_stride] = pick;
    c->tokens[(size_t)b * c->max_seq + c->st.n_known] =
        forced ? forced[(size_t)b * forced_stride] : pick;
  }
  if (out_logits) memcpy(out_logits, z, (size_t)B * V * sizeof(double));
  free(z);
}

int oracle_prefill(oracle_ctx *c, const int32_t *prompt, int32_t B, int32_t P,
                   const int32_t *forced_first, int32_t *out_token, double *out_logits) {
  if (!c || !prompt || B < 1 || P < 1) return -1;
  if (c->prefilled) return -3;
  if (B > c->max_batch || P + 1 > c->max_seq) return -4;
  for (int b = 0; b < B; ++b)
    for (int p = 0; p < P; ++p) {
      int32_t t = prompt[(size_t)b * P + p];
      if (t < 0 || t >= c->s.vocab) return -1;
      c->tokens[(size_t)b * c->max_seq + p] = t;
    }
  c->B = B;
  c->st.cycle = 1;
  int H = c->s.hidden, L = c->s.n_layers, lo = L - c->L_d;
  /* all prompt positions through all layers (Section 2.2: the prefill is the first pass of
   * the first cycle).  Rows are fed in causal chunks to bound memory; chunking does not
   * change any row's result because every row only looks at earlier positions. */
  const int chunk = 256;
  double *x = (double *)malloc((size_t)chunk * H * sizeof(double));
  double *last = (double *)malloc((size_t)B * H * sizeof(double));
  for (int b = 0; b < B; ++b) {
    for (int p0 = 0; p0 < P; p0 += chunk) {
      int R = P - p0 < chunk ? P - p0 : chunk;
      const int32_t *tok = c->tokens + (size_t)b * c->max_seq + p0;
      embed_rows(&c->s, &c->w, tok, R, x);
      /* base of Eq. 4's sum: the embedding, or (ExDy) the output of the encoding layers */
      double *base = (double *)malloc((size_t)R * H * sizeof(double));
      for (int l = 0; l < L; ++l) {
        if (l == c->L_e) memcpy(base, x, (size_t)R * H * sizeof(double));
        if (l == lo && c->literal_sum)
          for (size_t i = 0; i < (size_t)R * H; ++i) x[i] += base[i];
        layer_forward(&c->s, &c->layers[l], x, R, p0, oracle_k_cache(c, l, b),
                      oracle_v_cache(c, l, b));
      }
      free(base);
      if (p0 + R == P) memcpy(last + (size_t)b * H, x + (size_t)(R - 1) * H, (size_t)H * sizeof(double));
    }
  }
  for (int l = 0; l < L; ++l) { c->calls[l] += 1; c->rows[l] += P; }
  record_pass(c, 0, 0, P, 0, P);
  c->st.n_known = P;
  emit(c, last, forced_first, 1, out_token, 1, out_logits);
  c->st.lo_len = P; c->st.up_len = P; c->st.n_known = P + 1;
  c->st.slot = 1 % c->tau; c->st.n_emitted = 1;
  c->prefilled = 1;
  free(x); free(last);
  return 0;
}

/* One forward pass of the decode stage, full or short according to the slot.
 *
 * Every pass first takes the newest token's embedding through the L_e encoding layers (none in
 * the paper's default E0Dy setting) and keeps the result, h_enc, for that position: it is the
 * input of the decoding layers in a short pass (Section 2.1: h_enc takes the place of h_emb when
 * the encoding layers are reused too) and the input of the thinking layers when the position is
 * refilled.  lo_len is the number of positions with KV in the thinking layers [L_e, L - L_d). */
static int run_pass(oracle_ctx *c, const int32_t *forced, int forced_stride, int32_t *out_token,
                    int out_stride, double *out_logits) {
  if (c->st.n_known + 1 > c->max_seq) return -4;
  int B = c->B, H = c->s.hidden, L = c->s.n_layers, lo = L - c->L_d, Le = c->L_e;
  int newest = c->st.n_known - 1;          /* position of the token whose id we learnt last */
  double *xu = (double *)malloc((size_t)B * H * sizeof(double));   /* decoding-stack input */
  for (int b = 0; b < B; ++b)
    embed_rows(&c->s, &c->w, c->tokens + (size_t)b * c->max_seq + newest, 1, xu + (size_t)b * H);
  run_layers(c, 0, Le, xu, B, 1, newest);
  for (int b = 0; b < B; ++b)
    memcpy(c->h_enc + ((size_t)b * c->max_seq + newest) * H, xu + (size_t)b * H, (size_t)H * sizeof(double));
  if (c->st.slot != 0) {
    /* short pass: h_enc of the newest token goes straight into the decoding layers */
    record_pass(c, 2, 0, 0, newest, newest + 1);
  } else {
    /* full pass: every position the thinking layers have not seen yet (the tau-1 tokens of the
     * previous cycle plus the newest) goes through them together - this refills their KV -
     * and only the newest row continues upward */
    int p0 = c->st.lo_len, R = c->st.n_known - p0;
    double *x = (double *)malloc((size_t)B * R * H * sizeof(double));
    for (int b = 0; b < B; ++b)
      memcpy(x + (size_t)b * R * H, c->h_enc + ((size_t)b * c->max_seq + p0) * H, (size_t)R * H * sizeof(double));
    run_layers(c, Le, lo, x, B, R, p0);
    for (int b = 0; b < B; ++b) {
      double *dst = xu + (size_t)b * H;
      const double *think = x + ((size_t)b * R + (R - 1)) * H;
      const double *base = c->h_enc + ((size_t)b * c->max_seq + newest) * H;
      for (int i = 0; i < H; ++i) dst[i] = c->literal_sum ? base[i] + think[i] : think[i];
    }
    free(x);
    c->st.cycle += 1;
    record_pass(c, 1, p0, c->st.n_known, newest, newest + 1);
    c->st.lo_len = c->st.n_known;
  }
  run_layers(c, lo, L, xu, B, 1, newest);
  emit(c, xu, forced, forced_stride, out_token, out_stride, out_logits);
  free(xu);
  c->st.up_len = c->st.n_known;
  c->st.n_known += 1;
  c->st.slot = (c->st.slot + 1) % c->tau;
  c->st.n_emitted += 1;
  return 0;
}

int oracle_decode_cycle(oracle_ctx *c, int32_t max_new, int32_t *out_tokens, int32_t *n_out,
                        double *out_logits) {
  if (!c || !n_out || max_new < 0) return -1;
  if (!c->prefilled) return -3;
  int n = 0;
  size_t BV = (size_t)c->B * c->s.vocab;
  while (n < max_new) {
    int rc = run_pass(c, NULL, 0, out_tokens ? out_tokens + n : NULL, c->tau,
                      out_logits ? out_logits + (size_t)n * BV : NULL);
    if (rc) { *n_out = n; return rc; }
    ++n;
    if (c->st.slot == 0) break;            /* the cycle is complete */
  }
  *n_out = n;
  return 0;
}

int oracle_decode_forced(oracle_ctx *c, const int32_t *forced, int32_t n, double *out_logits,
                         int32_t *out_argmax) {
  if (!c || !forced || n < 0) return -1;
  if (!c->prefilled) return -3;
  size_t BV = (size_t)c->B * c->s.vocab;
  for (int i = 0; i < n; ++i) {
    int rc = run_pass(c, forced + i, n, out_argmax ? out_argmax + (size_t)i * c->B : NULL, 1,
                      out_logits ? out_logits + (size_t)i * BV : NULL);
    if (rc) return rc;
  }
  return 0;
}

int oracle_step_layers(oracle_ctx *c, int32_t l0, int32_t l1, double *hidden, int32_t B,
                       int32_t R, int32_t pos0) {
  if (!c || !hidden) return -1;
  if (l0 < 0 || l1 > c->s.n_layers || l0 > l1 || B < 1 || B > c->max_batch || R < 1 || pos0 < 0)
    return -1;
  if (pos0 + R > c->max_seq) return -4;
  run_layers(c, l0, l1, hidden, B, R, pos0);
  return 0;
}

int oracle_get_state(const oracle_ctx *c, oracle_state *s) {
  if (!c || !s) return -1;
  *s = c->st;
  return 0;
}

int oracle_get_trace(const oracle_ctx *c, oracle_pass_record *rec, int32_t max_records) {
  if (!c) return -1;
  int n = c->n_trace < max_records ? c->n_trace : max_records;
  if (rec && n > 0) memcpy(rec, c->trace, (size_t)n * sizeof *rec);
  return c->n_trace;
}

int oracle_get_layer_counters(const oracle_ctx *c, int64_t *calls, int64_t *rows) {
  if (!c) return -1;
  if (calls) memcpy(calls, c->calls, (size_t)c->s.n_layers * sizeof(int64_t));
  if (rows) memcpy(rows, c->rows, (size_t)c->s.n_layers * sizeof(int64_t));
  return 0;
}

/* ------------------------------------------------------------------ independent formulations */

/* The whole sequence tokens[0..n) through layers [l0, l1) as one causal chunk on fresh
 * caches; x [n][hidden] in/out. */
static void forward_no_reuse(const oracle_shape *s, const oracle_weights *w, int l0, int l1,
                             double *x, int n) {
  size_t kvd = (size_t)s->n_kv_heads * s->head_dim;
  double *kc = (double *)malloc((size_t)n * kvd * sizeof(double));
  double *vc = (double *)malloc((size_t)n * kvd * sizeof(double));
  for (int l = l0; l < l1; ++l) layer_forward(s, &w->layers[l], x, n, 0, kc, vc);
  free(kc); free(vc);
}

int oracle_vanilla_generate(const oracle_shape *shape, const oracle_weights *w, int32_t *tokens,
                            int32_t P, int32_t n_new, const int32_t *forced,
                            double *out_logits, int32_t *out_argmax) {
  if (!shape_ok(shape) || !w || !tokens || P < 1 || n_new < 0) return -1;
  int H = shape->hidden, V = shape->vocab;
  double *z = (double *)malloc((size_t)V * sizeof(double));
  for (int i = 0; i < n_new; ++i) {
    int n = P + i;
    double *x = (double *)malloc((size_t)n * H * sizeof(double));
    embed_rows(shape, w, tokens, n, x);
    forward_no_reuse(shape, w, 0, shape->n_layers, x, n);
    lm_head(shape, w, x + (size_t)(n - 1) * H, 1, z);
    int32_t pick = argmax_lowest(z, V);
    if (out_argmax) out_argmax[i] = pick;
    if (out_logits) memcpy(out_logits + (size_t)i * V, z, (size_t)V * sizeof(double));
    tokens[n] = forced ? forced[i] : pick;
    free(x);
  }
  free(z);
  return 0;
}

/* Eq. 3 with the cycle anchored at the last prompt position, as in Section 2.2's example:
 * m_p = 1 inside the prompt and wherever (p - (P-1)) mod tau == 0.  With P = 1 this is the
 * paper's p mod tau == 0. */
int oracle_anchor_mask(int32_t p, int32_t P, int32_t tau) {
  return (p < P) || ((p - (P - 1)) % tau == 0);
}

int oracle_masked_parallel_forward_exdy(const oracle_shape *shape, const oracle_weights *w,
                                        int32_t L_e, int32_t L_d, int32_t tau,
                                        const int32_t *tokens, int32_t n, int32_t P,
                                        int32_t literal_sum, double *out_logits) {
  if (!shape_ok(shape) || !w || !tokens || !out_logits) return -1;
  if (L_d < 1 || L_e < 0 || L_e + L_d > shape->n_layers || tau < 1 || P < 1 || n < P) return -1;
  int H = shape->hidden, L = shape->n_layers, lo = L - L_d;
  double *enc = (double *)malloc((size_t)n * H * sizeof(double));
  double *think = (double *)malloc((size_t)n * H * sizeof(double));
  embed_rows(shape, w, tokens, n, enc);                          /* h_emb */
  forward_no_reuse(shape, w, 0, L_e, enc, n);                    /* Eq. 1: h_enc (= h_emb when L_e = 0) */
  memcpy(think, enc, (size_t)n * H * sizeof(double));
  forward_no_reuse(shape, w, L_e, lo, think, n);                 /* Eq. 2: h_think */
  for (int p = 0; p < n; ++p) {
    int m = oracle_anchor_mask(p, P, tau);                        /* Eq. 3 */
    for (int i = 0; i < H; ++i) {
      size_t j = (size_t)p * H + i;
      if (!m) think[j] = enc[j];                                  /* Eq. 4 with h_enc in h_emb's place */
      else if (literal_sum) think[j] = enc[j] + think[j];
    }
  }
  forward_no_reuse(shape, w, lo, L, think, n);                   /* Eq. 5: decoding layers */
  lm_head(shape, w, think + (size_t)(P - 1) * H, n - (P - 1), out_logits);
  free(enc); free(think);
  return 0;
}

int oracle_masked_parallel_forward(const oracle_shape *shape, const oracle_weights *w,
                                   int32_t L_d, int32_t tau, const int32_t *tokens, int32_t n,
                                   int32_t P, int32_t literal_sum, double *out_logits) {
  return oracle_masked_parallel_forward_exdy(shape, w, 0, L_d, tau, tokens, n, P, literal_sum, out_logits);
}
