/* CPU oracle for the adaptive speculative-decoding iteration (AdaEAGLE).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, fp32 restatement of
 * what the decode iteration computes, written from the paper, and it exists so
 * that the CUDA library can be checked against something that is not itself.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may build or
 * call it.  It shares no code with the CUDA library.
 *
 * What is restated (paper passages in brackets):
 *   - Algorithm 1: prefill = first target pass with draft length 0; then
 *     verify -> predict length -> draft, until enough tokens are emitted.
 *   - Eq. 1 (verify): the target runs once over the pending token followed by
 *     the k draft tokens; k_accept = length of the longest draft prefix with no
 *     incorrect token (footnote to Section 3.1), plus one bonus token.
 *   - Eq. 2 (draft): the draft model emits k tokens one after another.
 *   - Eq. 3 (length predictor): MLP on [e ; f] of the last token of the
 *     validated prefix, f being the target's hidden state after the final
 *     normalisation (Section 3.2, and the pair ([e_j ; f_j], k^j) of Section 3.3).
 *     Two output forms: class logits with n = argmax + 1 (the "w/ Cls" variant
 *     of Section 4.3.2) and the scalar form Round -> clamp of Eq. 3.
 *   - EAGLE draft head (Section 2.2, Appendix A): reuses the target's embedding
 *     and LM head with one trainable block between them; consumes target
 *     features for verified positions and its own outputs for drafted ones.
 *   - Counters N_draft, N_target, N_waste and tau (caption of Table 2).
 *
 * The paper does not spell out the target's internals beyond "Llama family";
 * the layer is the standard pre-norm block: RMSNorm, rotary q/k (rotate-half
 * pairing), causal softmax attention, residual, RMSNorm, SwiGLU, residual.
 *
 * Parity pins (all in tests run without a GPU): the target forward is pinned
 * to an independent library implementation of the Llama block and to a
 * stock-op restatement; the KV-cache path to a cache-free recompute; the
 * emitted tokens to plain greedy decoding (lossless property); acceptance to
 * its definition on corrupted teacher-forced drafts; compaction to a fresh
 * prefill; the predictor to hand-computed cases; the counters to Table 2.
 * PARITY UNPINNED: how the draft head pairs features with tokens (feature of
 * position p with the embedding of token p+1, output = estimate of feature
 * p+1, no final norm).  The paper prints no example of it; only the block's
 * arithmetic is pinned (to the same library layer).
 *
 * Arithmetic: weights are bf16 bit patterns widened exactly to fp32; every
 * activation, cache entry and accumulator is fp32 (the paper's runs were FP32).
 * A dot product accumulates element k into partial sum (k mod 16) and adds the
 * 16 partial sums in a fixed tree, so a row's result never depends on how many
 * rows are processed together.  Argmax ties go to the lowest index.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rope_theta, rms_eps;
  int32_t ldlp_hidden, n_max;
  int32_t ldlp_mode;        /* 0: class logits, n = argmax + 1; 1: scalar, Round + clamp (Eq. 3) */
  int32_t ldlp_embed_shift; /* 0: e of the token whose hidden state is f (paper); 1: e of the bonus token */
  int32_t ldlp_blocks;      /* scalar form: number of residual blocks */
  int32_t k_min;            /* lower clamp of the scalar form (Eq. 3 prints 0; the loop needs >= 1) */
  float ddd_threshold;      /* < 0: AdaEAGLE-DDD (Section 4): log-probability threshold of the draft sequence; else off */
} orc_config;

typedef struct {
  const uint16_t *embed, *lm_head, *final_norm;
  const uint16_t *const *wq, *const *wk, *const *wv, *const *wo;
  const uint16_t *const *w_gate, *const *w_up, *const *w_down;
  const uint16_t *const *norm_attn, *const *norm_mlp;
  const uint16_t *eagle_fc;
  const uint16_t *e_wq, *e_wk, *e_wv, *e_wo, *e_gate, *e_up, *e_down, *e_norm_attn, *e_norm_mlp;
  const uint16_t *ldlp_w1, *ldlp_b1, *ldlp_w2, *ldlp_b2;
  const uint16_t *ldlp_wr, *ldlp_br; /* scalar form: [blocks][hid][hid], [blocks][hid] (may be NULL) */
} orc_weights;

typedef struct {
  orc_config c;
  orc_weights w;
} orc_model;

typedef struct {
  int cap;        /* positions allocated */
  int len;        /* committed tokens, the last one pending (not yet in the target cache) */
  int dlen;       /* draft-head cache rows that were computed from true target features */
  int32_t *tok;   /* [cap] committed tokens */
  float *feat;    /* [cap][d] target feature f_p (after the final norm) of every cached position */
  float *tk, *tv; /* [L][cap][d] target keys (rotated) and values */
  float *dk, *dv; /* [cap][d] draft-head keys and values */
  float *dfeat;   /* [n_max][d] draft-head outputs of the last draft call (step s -> row s-1) */
  int64_t n_target, n_draft, n_waste, n_tokens;
} orc_seq;

/* ------------------------------------------------------------------ basics */

static inline float bf(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* sum_k a[k] * b[k] with 16 interleaved partial sums and a fixed final tree */
static float dot16(const float *a, const float *b, int n) {
  float acc[16] = {0};
  int k = 0;
  for (; k + 16 <= n; k += 16)
    for (int i = 0; i < 16; ++i) acc[i] += a[k + i] * b[k + i];
  for (int i = 0; k + i < n; ++i) acc[i] += a[k + i] * b[k + i];
  for (int s = 8; s >= 1; s >>= 1)
    for (int i = 0; i < s; ++i) acc[i] += acc[i + s];
  return acc[0];
}

/* y[r][n] = sum_k x[r][k] * W[n][k]   (W: bf16 [N][K], row-major).
 * Rows are walked in blocks of 32 only so that x stays in cache; each output
 * element is the same dot16 whatever the block or the row count. */
static void linear(float *y, const float *x, const uint16_t *W, int R, int K, int N) {
  for (int r0 = 0; r0 < R; r0 += 32) {
    int r1 = r0 + 32 < R ? r0 + 32 : R;
#pragma omp parallel
    {
      float *wrow = (float *)malloc(sizeof(float) * (size_t)K);
#pragma omp for schedule(static)
      for (int n = 0; n < N; ++n) {
        const uint16_t *wn = W + (size_t)n * K;
        for (int k = 0; k < K; ++k) wrow[k] = bf(wn[k]);
        for (int r = r0; r < r1; ++r) y[(size_t)r * N + n] = dot16(x + (size_t)r * K, wrow, K);
      }
      free(wrow);
    }
  }
}

/* y = x / sqrt(mean(x^2) + eps) * g */
static void rmsnorm(float *y, const float *x, const uint16_t *g, int R, int d, float eps) {
  for (int r = 0; r < R; ++r) {
    const float *xr = x + (size_t)r * d;
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += (double)xr[i] * (double)xr[i];
    float inv = (float)(1.0 / sqrt(ss / d + (double)eps));
    for (int i = 0; i < d; ++i) y[(size_t)r * d + i] = (xr[i] * inv) * bf(g[i]);
  }
}

/* rotary embedding, rotate-half pairing (i, i + hd/2), angle = pos * theta^(-2i/hd) */
static void rope(float *x, int n_heads, int hd, int pos, float theta) {
  int half = hd / 2;
  for (int i = 0; i < half; ++i) {
    double ang = (double)pos * pow((double)theta, -2.0 * (double)i / (double)hd);
    float c = (float)cos(ang), s = (float)sin(ang);
    for (int h = 0; h < n_heads; ++h) {
      float *v = x + (size_t)h * hd;
      float a = v[i], b = v[i + half];
      v[i] = a * c - b * s;
      v[i + half] = b * c + a * s;
    }
  }
}

static int argmax_low(const float *v, int n) {
  int best = 0;
  for (int i = 1; i < n; ++i)
    if (v[i] > v[best]) best = i;
  return best;
}

static void top2(const float *v, int n, float *t1, float *t2) {
  int b = argmax_low(v, n);
  float s = -INFINITY;
  for (int i = 0; i < n; ++i)
    if (i != b && v[i] > s) s = v[i];
  *t1 = v[b];
  *t2 = s;
}

typedef struct {
  const uint16_t *wq, *wk, *wv, *wo, *wg, *wu, *wd, *na, *nm;
} layer_w;

/* One pre-norm decoder block over R rows at absolute positions pos0..pos0+R-1.
 * The rows' keys and values are first stored in the cache (kc, vc: [cap][d]);
 * row r then attends cache positions 0..pos0+r, which gives full attention to
 * the history and a causal mask inside the block. */
static void decoder_block(const orc_config *c, const layer_w *w, float *h, int R, int pos0,
                          float *kc, float *vc) {
  const int d = c->d_model, H = c->n_heads, hd = c->head_dim, F = c->d_ffn;
  float *u = (float *)malloc(sizeof(float) * (size_t)R * d);
  float *q = (float *)malloc(sizeof(float) * (size_t)R * d);
  float *a = (float *)malloc(sizeof(float) * (size_t)R * d);
  float *o = (float *)malloc(sizeof(float) * (size_t)R * d);
  float *g = (float *)malloc(sizeof(float) * (size_t)R * F);
  float *up = (float *)malloc(sizeof(float) * (size_t)R * F);

  rmsnorm(u, h, w->na, R, d, c->rms_eps);
  linear(q, u, w->wq, R, d, d);
  linear(kc + (size_t)pos0 * d, u, w->wk, R, d, d);
  linear(vc + (size_t)pos0 * d, u, w->wv, R, d, d);
  for (int r = 0; r < R; ++r) {
    rope(q + (size_t)r * d, H, hd, pos0 + r, c->rope_theta);
    rope(kc + (size_t)(pos0 + r) * d, H, hd, pos0 + r, c->rope_theta);
  }
  const float scale = 1.0f / sqrtf((float)hd);
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int r = 0; r < R; ++r) {
    for (int hh = 0; hh < H; ++hh) {
      int nk = pos0 + r + 1;
      float *s = (float *)malloc(sizeof(float) * (size_t)nk);
      const float *qv = q + (size_t)r * d + (size_t)hh * hd;
      float m = -INFINITY;
      for (int p = 0; p < nk; ++p) {
        s[p] = dot16(qv, kc + (size_t)p * d + (size_t)hh * hd, hd) * scale;
        if (s[p] > m) m = s[p];
      }
      double z = 0.0;
      for (int p = 0; p < nk; ++p) {
        s[p] = expf(s[p] - m);
        z += s[p];
      }
      float iz = (float)(1.0 / z);
      float *out = a + (size_t)r * d + (size_t)hh * hd;
      for (int i = 0; i < hd; ++i) out[i] = 0.0f;
      for (int p = 0; p < nk; ++p) {
        float pw = s[p] * iz;
        const float *vv = vc + (size_t)p * d + (size_t)hh * hd;
        for (int i = 0; i < hd; ++i) out[i] += pw * vv[i];
      }
      free(s);
    }
  }
  linear(o, a, w->wo, R, d, d);
  for (size_t i = 0; i < (size_t)R * d; ++i) h[i] += o[i];

  rmsnorm(u, h, w->nm, R, d, c->rms_eps);
  linear(g, u, w->wg, R, d, F);
  linear(up, u, w->wu, R, d, F);
  for (size_t i = 0; i < (size_t)R * F; ++i) {
    float x = g[i];
    g[i] = (x / (1.0f + expf(-x))) * up[i];
  }
  linear(o, g, w->wd, R, F, d);
  for (size_t i = 0; i < (size_t)R * d; ++i) h[i] += o[i];

  free(u); free(q); free(a); free(o); free(g); free(up);
}

static void embed_rows(const orc_model *m, const int32_t *tok, int R, float *h) {
  const int d = m->c.d_model;
  for (int r = 0; r < R; ++r)
    for (int i = 0; i < d; ++i) h[(size_t)r * d + i] = bf(m->w.embed[(size_t)tok[r] * d + i]);
}

static layer_w target_layer(const orc_model *m, int l) {
  layer_w w = {m->w.wq[l], m->w.wk[l], m->w.wv[l], m->w.wo[l], m->w.w_gate[l],
               m->w.w_up[l], m->w.w_down[l], m->w.norm_attn[l], m->w.norm_mlp[l]};
  return w;
}

/* Target pass over R tokens at positions pos0.. : fills the caches (k, v:
 * [L][cap][d]) and writes the post-final-norm features f (R x d). */
static void target_rows(const orc_model *m, const int32_t *tok, int R, int pos0, float *k, float *v,
                        int cap, float *f) {
  const int d = m->c.d_model;
  float *h = (float *)malloc(sizeof(float) * (size_t)R * d);
  embed_rows(m, tok, R, h);
  for (int l = 0; l < m->c.n_layers; ++l) {
    layer_w w = target_layer(m, l);
    decoder_block(&m->c, &w, h, R, pos0, k + (size_t)l * cap * d, v + (size_t)l * cap * d);
  }
  rmsnorm(f, h, m->w.final_norm, R, d, m->c.rms_eps);
  free(h);
}

/* Draft-head pass over R positions pos0.. : row r pairs the feature of position
 * pos0+r with the embedding of the token at position pos0+r+1 (next_tok[r]);
 * x = fc([e ; f]); one decoder block over the head's own cache; the block's
 * output (no further norm) estimates the feature of position pos0+r+1. */
static void draft_rows(const orc_model *m, const int32_t *next_tok, const float *feat, int R, int pos0,
                       float *dk, float *dv, float *out) {
  const int d = m->c.d_model;
  float *cat = (float *)malloc(sizeof(float) * (size_t)R * 2 * d);
  for (int r = 0; r < R; ++r) {
    for (int i = 0; i < d; ++i) {
      cat[(size_t)r * 2 * d + i] = bf(m->w.embed[(size_t)next_tok[r] * d + i]);
      cat[(size_t)r * 2 * d + d + i] = feat[(size_t)r * d + i];
    }
  }
  linear(out, cat, m->w.eagle_fc, R, 2 * d, d);
  layer_w w = {m->w.e_wq, m->w.e_wk, m->w.e_wv, m->w.e_wo, m->w.e_gate,
               m->w.e_up, m->w.e_down, m->w.e_norm_attn, m->w.e_norm_mlp};
  decoder_block(&m->c, &w, out, R, pos0, dk, dv);
  free(cat);
}

/* ------------------------------------------------------------ public calls */

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

orc_model *orc_model_create(const orc_config *c, const orc_weights *w) {
  orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
  m->c = *c;
  m->w = *w;
  return m;
}

void orc_model_destroy(orc_model *m) { free(m); }

orc_seq *orc_seq_create(const orc_model *m, int capacity) {
  const size_t d = (size_t)m->c.d_model, L = (size_t)m->c.n_layers, cap = (size_t)capacity;
  orc_seq *s = (orc_seq *)calloc(1, sizeof(orc_seq));
  s->cap = capacity;
  s->tok = (int32_t *)calloc(cap, sizeof(int32_t));
  s->feat = (float *)calloc(cap * d, sizeof(float));
  s->tk = (float *)calloc(L * cap * d, sizeof(float));
  s->tv = (float *)calloc(L * cap * d, sizeof(float));
  s->dk = (float *)calloc(cap * d, sizeof(float));
  s->dv = (float *)calloc(cap * d, sizeof(float));
  s->dfeat = (float *)calloc((size_t)(m->c.n_max > 0 ? m->c.n_max : 1) * d, sizeof(float));
  return s;
}

void orc_seq_destroy(orc_seq *s) {
  if (!s) return;
  free(s->tok); free(s->feat); free(s->tk); free(s->tv); free(s->dk); free(s->dv); free(s->dfeat);
  free(s);
}

/* Algorithm 1, first pass (draft length 0): the target reads the m prompt
 * tokens and yields the first new token.  Returns that token, or -1. */
int orc_prefill(const orc_model *m, orc_seq *s, const int32_t *prompt, int mlen) {
  const int d = m->c.d_model, V = m->c.vocab;
  if (mlen < 1 || mlen + 1 > s->cap) return -1;
  memcpy(s->tok, prompt, sizeof(int32_t) * (size_t)mlen);
  target_rows(m, prompt, mlen, 0, s->tk, s->tv, s->cap, s->feat);
  float *logits = (float *)malloc(sizeof(float) * (size_t)V);
  linear(logits, s->feat + (size_t)(mlen - 1) * d, m->w.lm_head, 1, d, V);
  s->tok[mlen] = argmax_low(logits, V);
  free(logits);
  s->len = mlen + 1;
  s->dlen = 0;
  s->n_target = s->n_draft = s->n_waste = s->n_tokens = 0;
  return s->tok[mlen];
}

/* Eq. 3.  Input [e ; f] of position len-2: the last token of the validated
 * prefix (the token before the pending bonus token) and the target feature at
 * that same position.  z_out (optional) receives the n_max class logits
 * (mode 0) or the scalar in z_out[0] (mode 1).  Returns the draft length. */
int orc_ldlp(const orc_model *m, const orc_seq *s, float *z_out) {
  const orc_config *c = &m->c;
  const int d = c->d_model, hid = c->ldlp_hidden;
  const int p = s->len - 2;
  if (p < 0) return -1;
  float *x = (float *)malloc(sizeof(float) * (size_t)2 * d);
  float *h = (float *)malloc(sizeof(float) * (size_t)hid);
  float *t = (float *)malloc(sizeof(float) * (size_t)hid);
  float z[64];
  const int etok = s->tok[p + (c->ldlp_embed_shift ? 1 : 0)];
  for (int i = 0; i < d; ++i) {
    x[i] = bf(m->w.embed[(size_t)etok * d + i]);
    x[d + i] = s->feat[(size_t)p * d + i];
  }
  linear(h, x, m->w.ldlp_w1, 1, 2 * d, hid);
  for (int i = 0; i < hid; ++i) {
    float v = h[i] + bf(m->w.ldlp_b1[i]);
    h[i] = v > 0.0f ? v : 0.0f;
  }
  int n;
  if (c->ldlp_mode == 0) {
    linear(z, h, m->w.ldlp_w2, 1, hid, c->n_max);
    for (int i = 0; i < c->n_max; ++i) z[i] += bf(m->w.ldlp_b2[i]);
    n = argmax_low(z, c->n_max) + 1;
    if (z_out) memcpy(z_out, z, sizeof(float) * (size_t)c->n_max);
  } else {
    /* residual blocks h += ReLU(W h + b), then a linear map to one scalar */
    for (int b = 0; b < c->ldlp_blocks; ++b) {
      linear(t, h, m->w.ldlp_wr + (size_t)b * hid * hid, 1, hid, hid);
      for (int i = 0; i < hid; ++i) {
        float v = t[i] + bf(m->w.ldlp_br[(size_t)b * hid + i]);
        h[i] += v > 0.0f ? v : 0.0f;
      }
    }
    linear(z, h, m->w.ldlp_w2, 1, hid, 1);
    z[0] += bf(m->w.ldlp_b2[0]);
    float kbar = rintf(z[0]); /* round half to even */
    float lo = (float)c->k_min, hi = (float)c->n_max;
    float kk = kbar < lo ? lo : (kbar > hi ? hi : kbar);
    n = (int)kk;
    if (z_out) z_out[0] = z[0];
  }
  free(x); free(h); free(t);
  return n;
}

/* Eq. 2.  First the head is brought up to date on the positions verified since
 * its last true-feature row (dlen .. len-2), using target features; the last of
 * those rows yields draft token 1.  Steps 2..n feed the head its own output.
 * forced (optional, n entries) replaces each drafted token after it is computed
 * (teacher forcing); draft_out receives the n tokens that enter the verify;
 * top1/top2 (optional, n entries) the two largest draft logits of each step. */
/* log of the softmax probability of logit `t` among the V logits (sums in double) */
static float log_prob_of(const float *logits, int V, int t) {
  float mx = logits[0];
  for (int i = 1; i < V; ++i) mx = logits[i] > mx ? logits[i] : mx;
  double sum = 0.0;
  for (int i = 0; i < V; ++i) sum += exp((double)logits[i] - (double)mx);
  return (float)((double)logits[t] - ((double)mx + log(sum)));
}

/* Draft with the combined stopping rule of Section 4 (AdaEAGLE-DDD): the head keeps drafting past the
 * predicted length n while the log-probability of the draft sequence so far (the sum of the log softmax
 * probabilities of its tokens) has not fallen below the threshold; it stops as soon as both hold, step >= n and
 * log-probability < threshold, and in any case at n_max tokens or at the cache capacity.  With ddd = 0
 * exactly n tokens are drafted.  logp_out (optional) receives the running log-probability after each token,
 * n_used the number of tokens drafted. */
static int draft_impl(const orc_model *m, orc_seq *s, int n, int ddd, const int32_t *forced, int32_t *draft_out,
                      float *top1, float *top2v, float *logp_out, int32_t *n_used) {
  const int d = m->c.d_model, V = m->c.vocab;
  const int j = s->len - 1; /* index of the pending token */
  if (n < 1 || n > m->c.n_max || j + n + 2 > s->cap) return -1;
  int n_lim = n;
  if (ddd) {
    n_lim = m->c.n_max;
    if (j + n_lim + 2 > s->cap) n_lim = s->cap - j - 2;
  }
  float seq_logp = 0.0f;
  float *logits = (float *)malloc(sizeof(float) * (size_t)V);
  const int R = j - s->dlen; /* catch-up rows: positions dlen .. j-1 */
  if (R < 1) { free(logits); return -2; }
  float *out = (float *)malloc(sizeof(float) * (size_t)(R > 1 ? R : 1) * d);
  draft_rows(m, s->tok + s->dlen + 1, s->feat + (size_t)s->dlen * d, R, s->dlen, s->dk, s->dv, out);
  s->dlen = j;
  memcpy(s->dfeat, out + (size_t)(R - 1) * d, sizeof(float) * (size_t)d);
  free(out);
  int made = 0;
  for (int step = 1; step <= n_lim; ++step) {
    float *fh = s->dfeat + (size_t)(step - 1) * d; /* estimate of the feature of position j+step-1 */
    if (step > 1) {
      /* position j+step-2: own feature of that position + embedding of draft token step-1 */
      draft_rows(m, &draft_out[step - 2], s->dfeat + (size_t)(step - 2) * d, 1, j + step - 2, s->dk,
                 s->dv, fh);
    }
    linear(logits, fh, m->w.lm_head, 1, d, V);
    int t = argmax_low(logits, V);
    if (top1 && top2v) top2(logits, V, &top1[step - 1], &top2v[step - 1]);
    draft_out[step - 1] = forced ? forced[step - 1] : t;
    made = step;
    if (ddd || logp_out) {
      seq_logp += log_prob_of(logits, V, draft_out[step - 1]);
      if (logp_out) logp_out[step - 1] = seq_logp;
    }
    if (ddd && step >= n && seq_logp < m->c.ddd_threshold) break;
  }
  if (n_used) *n_used = made;
  free(logits);
  return 0;
}

int orc_draft(const orc_model *m, orc_seq *s, int n, const int32_t *forced, int32_t *draft_out,
              float *top1, float *top2v) {
  return draft_impl(m, s, n, 0, forced, draft_out, top1, top2v, NULL, NULL);
}

/* as orc_draft, with the stopping rule of the model's configuration (ddd_threshold < 0: AdaEAGLE-DDD) */
int orc_draft_dyn(const orc_model *m, orc_seq *s, int n, const int32_t *forced, int32_t *draft_out,
                  float *top1, float *top2v, float *logp_out, int32_t *n_used) {
  return draft_impl(m, s, n, m->c.ddd_threshold < 0.0f, forced, draft_out, top1, top2v, logp_out, n_used);
}

/* Eq. 1, forward part.  Rows: the pending token then the n draft tokens, at
 * positions j..j+n.  target_tok[i] = argmax of the logits of row i.  logits
 * (optional) receives all (n+1) x V logits; top1/top2 (optional) the two
 * largest logits per row.  n = 0 is plain autoregressive decoding. */
int orc_verify(const orc_model *m, orc_seq *s, const int32_t *draft, int n, int32_t *target_tok,
               float *logits_out, float *top1, float *top2v) {
  const int d = m->c.d_model, V = m->c.vocab;
  const int j = s->len - 1;
  if (n < 0 || j + n + 2 > s->cap) return -1; /* up to n + 1 new tokens must fit the token array */
  const int R = n + 1;
  int32_t *rows = (int32_t *)malloc(sizeof(int32_t) * (size_t)R);
  rows[0] = s->tok[j];
  for (int i = 0; i < n; ++i) rows[i + 1] = draft[i];
  target_rows(m, rows, R, j, s->tk, s->tv, s->cap, s->feat + (size_t)j * d);
  float *logits = logits_out ? logits_out : (float *)malloc(sizeof(float) * (size_t)R * V);
  linear(logits, s->feat + (size_t)j * d, m->w.lm_head, R, d, V);
  for (int i = 0; i < R; ++i) {
    target_tok[i] = argmax_low(logits + (size_t)i * V, V);
    if (top1 && top2v) top2(logits + (size_t)i * V, V, &top1[i], &top2v[i]);
  }
  if (!logits_out) free(logits);
  free(rows);
  return 0;
}

/* Eq. 1, decision part, and the state update that follows.  k_accept = longest
 * draft prefix whose every token equals the target's choice at the row before
 * it; the bonus token is the target's choice after that prefix.  emitted gets
 * the k_accept accepted drafts then the bonus.  The target cache keeps rows
 * j..j+k_accept; the draft cache keeps only its true-feature rows.
 * Returns k_accept. */
int orc_accept(const orc_model *m, orc_seq *s, const int32_t *draft, const int32_t *target_tok, int n,
               int32_t *emitted, int32_t *n_emitted) {
  (void)m;
  const int j = s->len - 1;
  int k = 0;
  while (k < n && draft[k] == target_tok[k]) ++k;
  for (int i = 0; i < k; ++i) emitted[i] = draft[i];
  emitted[k] = target_tok[k];
  for (int i = 0; i <= k; ++i) s->tok[j + 1 + i] = emitted[i];
  s->len = j + k + 2;
  *n_emitted = k + 1;
  s->n_target += 1;
  s->n_draft += n;
  s->n_waste += n - k;
  s->n_tokens += k + 1;
  return k;
}

/* One iteration of the loop of Algorithm 1 in the order predict -> draft ->
 * verify -> accept.  n_forced < 0: use the predictor; n_forced = 0: no draft
 * (plain autoregressive step); otherwise a fixed length.  Lengths are clipped
 * so that the rows fit the cache.  Outputs are optional except emitted /
 * n_emitted.  Returns k_accept or a negative error. */
int orc_step(const orc_model *m, orc_seq *s, int n_forced, const int32_t *forced_draft,
             int32_t *emitted, int32_t *n_emitted, int32_t *n_used, int32_t *draft_out,
             int32_t *target_out, float *v_top1, float *v_top2, float *d_top1, float *d_top2,
             float *ldlp_z, float *d_logp) {
  int32_t draft[64], target[65];
  int n = n_forced;
  if (n < 0) n = orc_ldlp(m, s, ldlp_z);
  if (n < 0) return -1;
  const int j = s->len - 1;
  if (j + 2 > s->cap) return -2;
  if (j + n + 2 > s->cap) n = s->cap - j - 2;
  if (n >= 1) {
    int32_t made = n;
    if (orc_draft_dyn(m, s, n, forced_draft, draft, d_top1, d_top2, d_logp, &made)) return -3;
    n = made;
  }
  if (orc_verify(m, s, draft, n, target, NULL, v_top1, v_top2)) return -4;
  int k = orc_accept(m, s, draft, target, n, emitted, n_emitted);
  if (n_used) *n_used = n;
  if (draft_out) memcpy(draft_out, draft, sizeof(int32_t) * (size_t)n);
  if (target_out) memcpy(target_out, target, sizeof(int32_t) * (size_t)(n + 1));
  return k;
}

/* Label of Section 3.3 / the draft-length oracle of Section 2.3 for the current state: draft as many tokens as
 * allowed (n_max, or what the cache still holds), verify them, and return the length of the longest prefix of the
 * draft that the target confirms -- the optimal draft length for this iteration.  Nothing is committed: the
 * sequence is left as it was (the draft head's rows of true features are recomputed identically by the next
 * draft, the target's rows are overwritten by the next verify).  draft_out / target_out / n_out (optional) receive
 * the drafted tokens, the target's choices after each row, and the draft length. */
int orc_label(const orc_model *m, orc_seq *s, int32_t *draft_out, int32_t *target_out, int32_t *n_out) {
  int32_t draft[64], target[65];
  const int j = s->len - 1;
  int n = m->c.n_max;
  if (j + n + 2 > s->cap) n = s->cap - j - 2;
  if (n < 1) return 0;
  const int dlen0 = s->dlen;
  if (draft_impl(m, s, n, 0, NULL, draft, NULL, NULL, NULL, NULL)) return -1;
  if (orc_verify(m, s, draft, n, target, NULL, NULL, NULL)) return -2;
  s->dlen = dlen0;
  if (draft_out) memcpy(draft_out, draft, sizeof(int32_t) * (size_t)n);
  if (target_out) memcpy(target_out, target, sizeof(int32_t) * (size_t)(n + 1));
  if (n_out) *n_out = n;
  int k = 0;
  while (k < n && draft[k] == target[k]) ++k;
  return k;
}

/* Roll a sequence back to an earlier state of itself: the first `len` committed tokens stay (the last of them
 * pending again) and the draft head keeps its first `dlen` true-feature rows.  Cache rows, features and tokens past
 * those lengths are left in place as garbage; every later pass overwrites the rows it reads (dlen <= len - 2: the
 * row of position len - 2 yields the first draft token, so the next draft computes it).  Counters restart at
 * zero.  Used to run several continuations from one prefilled prompt. */
int orc_rewind(orc_seq *s, int len, int dlen) {
  if (len < 1 || len > s->len || dlen < 0 || dlen > s->dlen || dlen > len - 2) return -1;
  s->len = len;
  s->dlen = dlen;
  s->n_target = s->n_draft = s->n_waste = s->n_tokens = 0;
  return 0;
}

/* Cache-free recompute: the target reads tokens[0..len) from scratch and
 * returns the features (len x d, optional) and the logits of the last row
 * (optional).  Used as brute force against the cached path. */
int orc_forward_nocache(const orc_model *m, const int32_t *tokens, int len, float *feat_out,
                        float *logits_last) {
  const size_t d = (size_t)m->c.d_model, L = (size_t)m->c.n_layers;
  float *k = (float *)calloc(L * (size_t)len * d, sizeof(float));
  float *v = (float *)calloc(L * (size_t)len * d, sizeof(float));
  float *f = (float *)malloc(sizeof(float) * (size_t)len * d);
  target_rows(m, tokens, len, 0, k, v, len, f);
  if (feat_out) memcpy(feat_out, f, sizeof(float) * (size_t)len * d);
  if (logits_last) linear(logits_last, f + (size_t)(len - 1) * d, m->w.lm_head, 1, (int)d, m->c.vocab);
  free(k); free(v); free(f);
  return 0;
}

/* Draft head alone on given rows (no sequence state): for pinning the head's
 * arithmetic.  feat: R x d, next_tok: R, caches dk/dv: [pos0+R][d]. */
int orc_draft_rows(const orc_model *m, const int32_t *next_tok, const float *feat, int R, int pos0,
                   float *dk, float *dv, float *out) {
  draft_rows(m, next_tok, feat, R, pos0, dk, dv, out);
  return 0;
}

/* ------------------------------------------------------------- inspection */

int orc_seq_len(const orc_seq *s) { return s->len; }
int orc_seq_dlen(const orc_seq *s) { return s->dlen; }
const int32_t *orc_seq_tokens(const orc_seq *s) { return s->tok; }
const float *orc_seq_features(const orc_seq *s) { return s->feat; }
const float *orc_seq_draft_features(const orc_seq *s) { return s->dfeat; }
const float *orc_seq_target_k(const orc_seq *s) { return s->tk; }
const float *orc_seq_target_v(const orc_seq *s) { return s->tv; }
void orc_seq_counters(const orc_seq *s, int64_t out[4]) {
  out[0] = s->n_target; out[1] = s->n_draft; out[2] = s->n_waste; out[3] = s->n_tokens;
}

/* tau of Table 2: accepted tokens per target pass */
double orc_tau(int64_t n_draft, int64_t n_target, int64_t n_waste) {
  return 1.0 + (double)(n_draft - n_waste) / (double)n_target;
}
