/*
 * CPU checker for the verification step of Aggressive Decoding (arXiv 2205.10350).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * library is compared against.  It shares no code with that library, and the library
 * never calls it.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may build or run it.
 *
 * What it computes
 *   - a post-LayerNorm encoder-decoder Transformer (paper Section 2; sizes from
 *     Sections 4.1.1 and 4.2.1), single sentence at a time, plain loops;
 *   - greedy autoregressive decoding (Section 2, the arg-max recurrence after Eq. 1);
 *   - the block verification forward: all positions of a drafted block scored in one
 *     teacher-forced pass on top of a key/value cache of the accepted prefix (Eq. 1, Eq. 3,
 *     Eq. 6, Eq. 7);
 *   - the bifurcation / acceptance rule (Section 3.1.1; the definition of c and the accepted
 *     block after Eq. 7) including the no-mismatch case and truncation at [EOS];
 *   - Algorithm 1 (input-guided mode) with its suffix-match rule;
 *   - the generalized mode loop of Section 3.2 with a non-autoregressive drafter forward
 *     (Section 3.2.1: prefix followed by k [MASK] inputs, bidirectional attention, no cache).
 *
 * Precision: ORC_REAL (float unless overridden with -DORC_REAL=double).  Every dot product is
 * accumulated in a fixed ascending order of the contraction index, so the score of a position
 * does not depend on how many other positions share the pass.  Build with contraction off
 * (-ffp-contract=off) so that this holds in vectorised code too.
 *
 * Parity pins (tests/test_oracle_*.py): brute-force attention, closed forms for LayerNorm and the
 * positional table, identity/one-hot linear maps, cross-checks of each sub-block against library
 * routines, incremental == full recompute bit for bit, block == single step bit for bit,
 * draft-verify == greedy for arbitrary drafts, iteration-count closed forms, the block shapes of
 * the paper's worked case study.  The text outputs of the paper's trained models are
 * "parity unpinned": weights and data are not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef ORC_REAL
#define ORC_REAL float
#endif
typedef ORC_REAL real;

typedef struct {
  int d_model, n_heads, d_ffn, vocab, n_enc, n_dec, max_pos;
  int bos, pad, eos, mask;
  double ln_eps;
} orc_cfg;

typedef struct { const real *Wq, *bq, *Wk, *bk, *Wv, *bv, *Wo, *bo; } attn_w;
typedef struct { const real *g, *b; } ln_w;
typedef struct { const real *W1, *b1, *W2, *b2; } ffn_w;
typedef struct { attn_w self; ln_w ln1; ffn_w ffn; ln_w ln2; } enc_layer;
typedef struct { attn_w self; ln_w ln1; attn_w cross; ln_w ln2; ffn_w ffn; ln_w ln3; } dec_layer;

typedef struct {
  orc_cfg cfg;
  const real* emb;   /* [V, d] shared by encoder input, decoder input and output projection */
  real* pe;          /* [max_pos, d] sinusoidal table */
  enc_layer* enc;
  dec_layer* dec;
} orc_model;

/* Per-sentence decoding state: encoder memory projected to per-layer cross K/V, and the
 * self-attention K/V cache of the accepted prefix. */
typedef struct {
  const orc_model* m;
  int S;             /* source length */
  int cap;           /* cache capacity in positions */
  int len;           /* accepted-prefix length = number of cached positions */
  real* mem;         /* [S, d] encoder output */
  real* ck;          /* [n_dec][S, d] */
  real* cv;
  real* sk;          /* [n_dec][cap, d] */
  real* sv;
} orc_state;

/* ------------------------------------------------------------------------------------------ */
/* Elementary maps                                                                            */
/* ------------------------------------------------------------------------------------------ */

/* y[M,out] = x[M,in] W[in,out] + b.  For each output element the sum runs over the input index in
 * ascending order, starting from the bias. */
void orc_linear(const real* x, const real* W, const real* b, real* y, int M, int in, int out) {
  const int BL = 64;
  int nblk = (out + BL - 1) / BL;
#pragma omp parallel for collapse(2) schedule(static)
  for (int m = 0; m < M; ++m) {
    for (int jb = 0; jb < nblk; ++jb) {
      int j0 = jb * BL, j1 = j0 + BL < out ? j0 + BL : out;
      real* yr = y + (size_t)m * out;
      const real* xr = x + (size_t)m * in;
      for (int j = j0; j < j1; ++j) yr[j] = b ? b[j] : (real)0;
      for (int i = 0; i < in; ++i) {
        real xi = xr[i];
        const real* wr = W + (size_t)i * out;
        for (int j = j0; j < j1; ++j) yr[j] += xi * wr[j];
      }
    }
  }
}

/* LayerNorm over the last dimension with biased variance: y = g (x - mean) / sqrt(var + eps) + b. */
void orc_layernorm(const real* x, const real* g, const real* b, real* y, int M, int d, double eps) {
  for (int m = 0; m < M; ++m) {
    const real* xr = x + (size_t)m * d;
    real* yr = y + (size_t)m * d;
    real mean = 0;
    for (int i = 0; i < d; ++i) mean += xr[i];
    mean /= (real)d;
    real var = 0;
    for (int i = 0; i < d; ++i) { real t = xr[i] - mean; var += t * t; }
    var /= (real)d;
    real inv = (real)1 / (real)sqrt((double)var + eps);
    for (int i = 0; i < d; ++i) yr[i] = g[i] * ((xr[i] - mean) * inv) + b[i];
  }
}

/* Scaled dot-product attention for one head-split projection set.
 * q [Mq, d], k/v [Mk, d] (all heads side by side).  Query i may attend keys 0 .. limit[i]-1.
 * out [Mq, d].  Scores are q.k / sqrt(dh); softmax subtracts the row maximum. */
void orc_attention(const real* q, const real* k, const real* v, const int* limit, real* out,
                   int Mq, int Mk, int d, int H) {
  int dh = d / H;
  real scale = (real)1 / (real)sqrt((double)dh);
#pragma omp parallel for collapse(2) schedule(static)
  for (int i = 0; i < Mq; ++i) {
    for (int h = 0; h < H; ++h) {
      int n = limit[i] < Mk ? limit[i] : Mk;
      real* p = (real*)malloc(sizeof(real) * (size_t)(n > 0 ? n : 1));
      const real* qi = q + (size_t)i * d + h * dh;
      real mx = -INFINITY;
      for (int j = 0; j < n; ++j) {
        const real* kj = k + (size_t)j * d + h * dh;
        real s = 0;
        for (int c = 0; c < dh; ++c) s += qi[c] * kj[c];
        s *= scale;
        p[j] = s;
        if (s > mx) mx = s;
      }
      real den = 0;
      for (int j = 0; j < n; ++j) { p[j] = (real)exp((double)(p[j] - mx)); den += p[j]; }
      real* o = out + (size_t)i * d + h * dh;
      for (int c = 0; c < dh; ++c) o[c] = 0;
      for (int j = 0; j < n; ++j) {
        real w = p[j] / den;
        const real* vj = v + (size_t)j * d + h * dh;
        for (int c = 0; c < dh; ++c) o[c] += w * vj[c];
      }
      free(p);
    }
  }
}

/* x[m,:] = emb[tok[m],:] * sqrt(d) + pe[pos0+m,:] */
static void embed(const orc_model* m, const int* tok, int M, int pos0, real* x) {
  int d = m->cfg.d_model;
  real sc = (real)sqrt((double)d);
  for (int r = 0; r < M; ++r) {
    const real* e = m->emb + (size_t)tok[r] * d;
    const real* p = m->pe + (size_t)(pos0 + r) * d;
    for (int i = 0; i < d; ++i) x[(size_t)r * d + i] = e[i] * sc + p[i];
  }
}

static void add_inplace(real* a, const real* b, size_t n) { for (size_t i = 0; i < n; ++i) a[i] += b[i]; }

static void ffn_block(const ffn_w* f, const real* x, real* y, int M, int d, int F) {
  real* h = (real*)malloc(sizeof(real) * (size_t)M * F);
  orc_linear(x, f->W1, f->b1, h, M, d, F);
  for (size_t i = 0; i < (size_t)M * F; ++i) h[i] = h[i] > 0 ? h[i] : (real)0;
  orc_linear(h, f->W2, f->b2, y, M, F, d);
  free(h);
}

/* ------------------------------------------------------------------------------------------ */
/* Model construction                                                                         */
/* ------------------------------------------------------------------------------------------ */

/* Sinusoidal positional table: PE(p, 2i) = sin(p / 10000^(2i/d)), PE(p, 2i+1) = cos(same). */
static void build_pe(real* pe, int max_pos, int d) {
  for (int p = 0; p < max_pos; ++p)
    for (int i = 0; i < d; i += 2) {
      double ang = (double)p / pow(10000.0, (double)i / (double)d);
      pe[(size_t)p * d + i] = (real)sin(ang);
      if (i + 1 < d) pe[(size_t)p * d + i + 1] = (real)cos(ang);
    }
}

static const real* take(const real** cur, size_t n) { const real* p = *cur; *cur += n; return p; }
static void take_attn(attn_w* a, const real** cur, int d) {
  a->Wq = take(cur, (size_t)d * d); a->bq = take(cur, d);
  a->Wk = take(cur, (size_t)d * d); a->bk = take(cur, d);
  a->Wv = take(cur, (size_t)d * d); a->bv = take(cur, d);
  a->Wo = take(cur, (size_t)d * d); a->bo = take(cur, d);
}
static void take_ln(ln_w* l, const real** cur, int d) { l->g = take(cur, d); l->b = take(cur, d); }
static void take_ffn(ffn_w* f, const real** cur, int d, int F) {
  f->W1 = take(cur, (size_t)d * F); f->b1 = take(cur, F);
  f->W2 = take(cur, (size_t)F * d); f->b2 = take(cur, d);
}

/* Number of reals the flat weight buffer must hold. */
size_t orc_weight_count(const orc_cfg* c) {
  size_t d = c->d_model, F = c->d_ffn, V = c->vocab;
  size_t attn = 4 * (d * d + d), ln = 2 * d, ffn = d * F + F + F * d + d;
  return V * d + (size_t)c->n_enc * (attn + ln + ffn + ln) + (size_t)c->n_dec * (attn + ln + attn + ln + ffn + ln);
}

/* flat: emb, then per encoder layer {self q,k,v,o (W,b each), ln1, ffn1, ffn2, ln2}, then per decoder
 * layer {self, ln1, cross, ln2, ffn1, ffn2, ln3}.  Every W is [in, out].  The buffer is borrowed. */
orc_model* orc_model_create(const orc_cfg* c, const real* flat) {
  orc_model* m = (orc_model*)calloc(1, sizeof(orc_model));
  m->cfg = *c;
  int d = c->d_model, F = c->d_ffn;
  const real* cur = flat;
  m->emb = take(&cur, (size_t)c->vocab * d);
  m->enc = (enc_layer*)calloc((size_t)(c->n_enc > 0 ? c->n_enc : 1), sizeof(enc_layer));
  m->dec = (dec_layer*)calloc((size_t)(c->n_dec > 0 ? c->n_dec : 1), sizeof(dec_layer));
  for (int l = 0; l < c->n_enc; ++l) {
    take_attn(&m->enc[l].self, &cur, d); take_ln(&m->enc[l].ln1, &cur, d);
    take_ffn(&m->enc[l].ffn, &cur, d, F); take_ln(&m->enc[l].ln2, &cur, d);
  }
  for (int l = 0; l < c->n_dec; ++l) {
    take_attn(&m->dec[l].self, &cur, d); take_ln(&m->dec[l].ln1, &cur, d);
    take_attn(&m->dec[l].cross, &cur, d); take_ln(&m->dec[l].ln2, &cur, d);
    take_ffn(&m->dec[l].ffn, &cur, d, F); take_ln(&m->dec[l].ln3, &cur, d);
  }
  m->pe = (real*)malloc(sizeof(real) * (size_t)c->max_pos * d);
  build_pe(m->pe, c->max_pos, d);
  return m;
}

void orc_model_destroy(orc_model* m) {
  if (!m) return;
  free(m->pe); free(m->enc); free(m->dec); free(m);
}

const real* orc_model_pe(const orc_model* m) { return m->pe; }

/* ------------------------------------------------------------------------------------------ */
/* Encoder                                                                                    */
/* ------------------------------------------------------------------------------------------ */

/* Encoder stack over one unpadded source of S tokens (so no padding mask is needed here; a
 * right-padded batch row gives the same result when its padding keys are masked out).
 * mem [S, d]. */
void orc_encode_memory(const orc_model* m, const int* src, int S, real* mem) {
  int d = m->cfg.d_model, H = m->cfg.n_heads, F = m->cfg.d_ffn;
  size_t n = (size_t)S * d;
  real *x = mem, *q = malloc(sizeof(real) * n), *k = malloc(sizeof(real) * n), *v = malloc(sizeof(real) * n);
  real *a = malloc(sizeof(real) * n), *t = malloc(sizeof(real) * n);
  int* lim = malloc(sizeof(int) * (size_t)S);
  for (int i = 0; i < S; ++i) lim[i] = S;
  embed(m, src, S, 0, x);
  for (int l = 0; l < m->cfg.n_enc; ++l) {
    const enc_layer* L = &m->enc[l];
    orc_linear(x, L->self.Wq, L->self.bq, q, S, d, d);
    orc_linear(x, L->self.Wk, L->self.bk, k, S, d, d);
    orc_linear(x, L->self.Wv, L->self.bv, v, S, d, d);
    orc_attention(q, k, v, lim, a, S, S, d, H);
    orc_linear(a, L->self.Wo, L->self.bo, t, S, d, d);
    add_inplace(t, x, n);
    orc_layernorm(t, L->ln1.g, L->ln1.b, x, S, d, m->cfg.ln_eps);
    ffn_block(&L->ffn, x, t, S, d, F);
    add_inplace(t, x, n);
    orc_layernorm(t, L->ln2.g, L->ln2.b, x, S, d, m->cfg.ln_eps);
  }
  free(q); free(k); free(v); free(a); free(t); free(lim);
}

orc_state* orc_state_create(const orc_model* m, const int* src, int S, int cap) {
  orc_state* s = (orc_state*)calloc(1, sizeof(orc_state));
  int d = m->cfg.d_model, Ld = m->cfg.n_dec;
  s->m = m; s->S = S; s->cap = cap; s->len = 0;
  s->mem = malloc(sizeof(real) * (size_t)S * d);
  s->ck = malloc(sizeof(real) * (size_t)Ld * S * d);
  s->cv = malloc(sizeof(real) * (size_t)Ld * S * d);
  s->sk = calloc((size_t)Ld * cap * d, sizeof(real));
  s->sv = calloc((size_t)Ld * cap * d, sizeof(real));
  orc_encode_memory(m, src, S, s->mem);
  for (int l = 0; l < Ld; ++l) {
    const attn_w* c = &m->dec[l].cross;
    orc_linear(s->mem, c->Wk, c->bk, s->ck + (size_t)l * S * d, S, d, d);
    orc_linear(s->mem, c->Wv, c->bv, s->cv + (size_t)l * S * d, S, d, d);
  }
  return s;
}

void orc_state_destroy(orc_state* s) {
  if (!s) return;
  free(s->mem); free(s->ck); free(s->cv); free(s->sk); free(s->sv); free(s);
}

int orc_state_len(const orc_state* s) { return s->len; }
const real* orc_state_memory(const orc_state* s) { return s->mem; }
void orc_state_reset(orc_state* s) { s->len = 0; }

/* ------------------------------------------------------------------------------------------ */
/* Decoder                                                                                    */
/* ------------------------------------------------------------------------------------------ */

static void logits_from(const orc_model* m, const real* y, int M, real* logits) {
  int d = m->cfg.d_model, V = m->cfg.vocab;
#pragma omp parallel for schedule(static)
  for (int v = 0; v < V; ++v) {
    const real* e = m->emb + (size_t)v * d;
    for (int r = 0; r < M; ++r) {
      const real* yr = y + (size_t)r * d;
      real s = 0;
      for (int i = 0; i < d; ++i) s += yr[i] * e[i];
      logits[(size_t)r * V + v] = s;
    }
  }
}

/* Block forward on top of the cache (Eq. 1 applied to a block; Eq. 6 / Eq. 7 inputs).
 * tok[0..k-1] are the decoder inputs at positions len .. len+k-1.  Writes tentative K/V for those
 * positions into the cache and does not change len.  logits [k, V].  Returns 0, or -1 if the
 * block does not fit. */
int orc_decode_block(orc_state* s, const int* tok, int k, real* logits) {
  const orc_model* m = s->m;
  int d = m->cfg.d_model, H = m->cfg.n_heads, F = m->cfg.d_ffn, S = s->S, len = s->len;
  if (k < 1 || len + k > s->cap || len + k > m->cfg.max_pos) return -1;
  size_t n = (size_t)k * d;
  real *y = malloc(sizeof(real) * n), *q = malloc(sizeof(real) * n), *a = malloc(sizeof(real) * n), *t = malloc(sizeof(real) * n);
  int *lim = malloc(sizeof(int) * (size_t)k), *limx = malloc(sizeof(int) * (size_t)k);
  for (int i = 0; i < k; ++i) { lim[i] = len + i + 1; limx[i] = S; }
  embed(m, tok, k, len, y);
  for (int l = 0; l < m->cfg.n_dec; ++l) {
    const dec_layer* L = &m->dec[l];
    real* K = s->sk + (size_t)l * s->cap * d;
    real* Vv = s->sv + (size_t)l * s->cap * d;
    orc_linear(y, L->self.Wq, L->self.bq, q, k, d, d);
    orc_linear(y, L->self.Wk, L->self.bk, K + (size_t)len * d, k, d, d);
    orc_linear(y, L->self.Wv, L->self.bv, Vv + (size_t)len * d, k, d, d);
    orc_attention(q, K, Vv, lim, a, k, len + k, d, H);
    orc_linear(a, L->self.Wo, L->self.bo, t, k, d, d);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln1.g, L->ln1.b, y, k, d, m->cfg.ln_eps);

    orc_linear(y, L->cross.Wq, L->cross.bq, q, k, d, d);
    orc_attention(q, s->ck + (size_t)l * S * d, s->cv + (size_t)l * S * d, limx, a, k, S, d, H);
    orc_linear(a, L->cross.Wo, L->cross.bo, t, k, d, d);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln2.g, L->ln2.b, y, k, d, m->cfg.ln_eps);

    ffn_block(&L->ffn, y, t, k, d, F);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln3.g, L->ln3.b, y, k, d, m->cfg.ln_eps);
  }
  logits_from(m, y, k, logits);
  free(y); free(q); free(a); free(t); free(lim); free(limx);
  return 0;
}

/* Decoder over a whole token sequence with no cache.  causal != 0: position i sees 0..i (the
 * teacher-forced scorer of Eq. 1); causal == 0: every position sees all T (the drafter of
 * Section 3.2.1).  mem / S: that model's own encoder memory.  logits [T, V]. */
void orc_decode_full(const orc_model* m, const real* mem, int S, const int* tok, int T, int causal, real* logits) {
  int d = m->cfg.d_model, H = m->cfg.n_heads, F = m->cfg.d_ffn;
  size_t n = (size_t)T * d, ns = (size_t)S * d;
  real *y = malloc(sizeof(real) * n), *q = malloc(sizeof(real) * n), *k = malloc(sizeof(real) * n), *v = malloc(sizeof(real) * n);
  real *a = malloc(sizeof(real) * n), *t = malloc(sizeof(real) * n);
  real *ck = malloc(sizeof(real) * ns), *cv = malloc(sizeof(real) * ns);
  int *lim = malloc(sizeof(int) * (size_t)T), *limx = malloc(sizeof(int) * (size_t)T);
  for (int i = 0; i < T; ++i) { lim[i] = causal ? i + 1 : T; limx[i] = S; }
  embed(m, tok, T, 0, y);
  for (int l = 0; l < m->cfg.n_dec; ++l) {
    const dec_layer* L = &m->dec[l];
    orc_linear(y, L->self.Wq, L->self.bq, q, T, d, d);
    orc_linear(y, L->self.Wk, L->self.bk, k, T, d, d);
    orc_linear(y, L->self.Wv, L->self.bv, v, T, d, d);
    orc_attention(q, k, v, lim, a, T, T, d, H);
    orc_linear(a, L->self.Wo, L->self.bo, t, T, d, d);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln1.g, L->ln1.b, y, T, d, m->cfg.ln_eps);

    orc_linear(mem, L->cross.Wk, L->cross.bk, ck, S, d, d);
    orc_linear(mem, L->cross.Wv, L->cross.bv, cv, S, d, d);
    orc_linear(y, L->cross.Wq, L->cross.bq, q, T, d, d);
    orc_attention(q, ck, cv, limx, a, T, S, d, H);
    orc_linear(a, L->cross.Wo, L->cross.bo, t, T, d, d);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln2.g, L->ln2.b, y, T, d, m->cfg.ln_eps);

    ffn_block(&L->ffn, y, t, T, d, F);
    add_inplace(t, y, n);
    orc_layernorm(t, L->ln3.g, L->ln3.b, y, T, d, m->cfg.ln_eps);
  }
  logits_from(m, y, T, logits);
  free(y); free(q); free(k); free(v); free(a); free(t); free(ck); free(cv); free(lim); free(limx);
}

/* ------------------------------------------------------------------------------------------ */
/* Integer logic of the method                                                                */
/* ------------------------------------------------------------------------------------------ */

/* Greedy choice: the largest score, lowest id on ties.  Also reports the runner-up. */
void orc_top2(const real* logits, int V, int* id1, real* v1, int* id2, real* v2) {
  int a = 0, b = -1;
  for (int v = 1; v < V; ++v) {
    if (logits[v] > logits[a]) { b = a; a = v; }
    else if (b < 0 || logits[v] > logits[b]) b = v;
  }
  *id1 = a; *v1 = logits[a];
  if (id2) *id2 = b;
  if (v2) *v2 = b >= 0 ? logits[b] : -INFINITY;
}

/* Relaxed verification of Section 3.2.3 (GAD++) on the scores of one position.  The drafted token is kept
 * when both conditions of the section hold, otherwise the greedy choice of Eq. 7 is taken:
 *   Eq. 8:  log P(draft) >= log P(beta-th ranked token)
 *   Eq. 9:  log P(top-1) - log P(draft) <= tau
 * log P = score - log(sum of exp(scores)); the normaliser is the same for every token of the position, so both
 * conditions are evaluated on the scores themselves.  beta >= 1; a negative draft (sentinel) never qualifies.
 * Outputs (each optional): met = 1 when the draft was kept; top_margin = top-1 minus top-2 score;
 * decision_margin = how far the scores are from flipping either condition: min(|score(draft) - u_beta|,
 * |tau - (top1 - score(draft))|), u_beta being the beta-th largest score among the OTHER tokens (the draft passes
 * Eq. 8 exactly when its score is >= u_beta); +inf where there is nothing to decide. */
static int cmp_desc(const void* a, const void* b) {
  const real x = *(const real*)a, y = *(const real*)b;
  return (x < y) - (x > y);
}
int orc_relaxed_choice(const real* logits, int V, int draft, int beta, double tau, int* met, real* top_margin,
                       real* decision_margin) {
  int top, second; real v1, v2;
  orc_top2(logits, V, &top, &v1, &second, &v2);
  if (top_margin) *top_margin = v1 - v2;
  if (met) *met = 0;
  if (decision_margin) *decision_margin = INFINITY;
  if (draft < 0 || draft >= V || beta < 1) return top;
  real* sorted = malloc(sizeof(real) * (size_t)V);
  memcpy(sorted, logits, sizeof(real) * (size_t)V);
  qsort(sorted, (size_t)V, sizeof(real), cmp_desc);
  const real vd = logits[draft];
  const real ranked = sorted[(beta <= V ? beta : V) - 1];          /* score of the beta-th ranked token */
  const int in_top_beta = vd >= ranked;                            /* Eq. 8 */
  const int within_tau = (double)v1 - (double)vd <= tau;           /* Eq. 9 */
  if (decision_margin) {
    /* beta-th largest among the other tokens: drop one occurrence of the draft's own score from the ranking */
    real u = -INFINITY;
    int seen = 0, skipped = 0;
    for (int i = 0; i < V && seen < beta; ++i) {
      if (!skipped && sorted[i] == vd) { skipped = 1; continue; }
      u = sorted[i]; ++seen;
    }
    const real m_rank = seen < beta ? INFINITY : (real)fabs((double)vd - (double)u);
    const real m_tau = (real)fabs(tau - ((double)v1 - (double)vd));
    *decision_margin = m_rank < m_tau ? m_rank : m_tau;
  }
  free(sorted);
  if (in_top_beta && within_tau) { if (met) *met = 1; return draft; }
  return top;
}

/* Acceptance rule.  pred[0..k-1] are the verifier's greedy choices, draft[0..k-1] the drafted tokens
 * they are compared with (draft[i] < 0 is a sentinel that matches nothing).
 *   c = first i with pred[i] != draft[i]  ->  n = c + 1   (the bifurcation token is accepted)
 *   no mismatch                            ->  n = k
 *   an [EOS] among pred[0..n-1] at index e ->  n = e + 1 and *finished = 1
 * Always 1 <= n <= k. */
int orc_accept(const int* pred, const int* draft, int k, int eos, int* finished) {
  int n = k;
  for (int i = 0; i < k; ++i)
    if (draft[i] < 0 || pred[i] != draft[i]) { n = i + 1; break; }
  int fin = 0;
  for (int i = 0; i < n; ++i)
    if (pred[i] == eos) { n = i + 1; fin = 1; break; }
  if (finished) *finished = fin;
  return n;
}

/* Suffix match of Algorithm 1, line 3.  o[0..j] (o[0] = BOS) is the output so far, x[0..n] is the
 * source with x[0] = BOS (the appended [PAD] is not part of the searched text).  For q = 0, 1, 2, ...
 * (q <= j) count the end positions i (q <= i <= n) with o[j-q..j] == x[i-q..i]:
 *   exactly one  -> return that i;   none -> return -1;   several -> try a longer suffix.
 * If the suffix cannot be made longer and is still ambiguous, return -1. */
int orc_suffix_match(const int* o, int j, const int* x, int n) {
  for (int q = 0; q <= j; ++q) {
    int count = 0, where = -1;
    for (int i = q; i <= n; ++i) {
      int ok = 1;
      for (int t = 0; t <= q; ++t)
        if (o[j - t] != x[i - t]) { ok = 0; break; }
      if (ok) { ++count; where = i; }
    }
    if (count == 1) return where;
    if (count == 0) return -1;
  }
  return -1;
}

/* One verification call on the state: feed (last, draft[0..k-2]), take greedy choices, apply the
 * acceptance rule.  pred [k], margin [k] (top-1 minus top-2 score), logits_out optional [k, V].
 * Does not commit.  Returns n (>= 1) or a negative error. */
int orc_verify_block(orc_state* s, int last, const int* draft, int k, int* pred, real* margin,
                     real* logits_out, int* finished) {
  int V = s->m->cfg.vocab;
  int* tok = malloc(sizeof(int) * (size_t)k);
  real* lg = logits_out ? logits_out : malloc(sizeof(real) * (size_t)k * V);
  tok[0] = last;
  for (int i = 1; i < k; ++i) tok[i] = draft[i - 1] >= 0 ? draft[i - 1] : s->m->cfg.pad;
  int rc = orc_decode_block(s, tok, k, lg);
  if (rc == 0) {
    for (int i = 0; i < k; ++i) {
      real v1, v2; int i2;
      orc_top2(lg + (size_t)i * V, V, &pred[i], &v1, &i2, &v2);
      if (margin) margin[i] = v1 - v2;
    }
    rc = orc_accept(pred, draft, k, s->m->cfg.eos, finished);
  }
  free(tok);
  if (!logits_out) free(lg);
  return rc;
}

/* The same call with the relaxed verification of Section 3.2.3: pred[i] is the drafted token where it meets
 * the top-beta / tau requirement and the greedy choice elsewhere; the acceptance rule is unchanged (the first
 * position whose verified token differs from the draft is the bifurcation).  met [k], margin [k] (top-1 minus
 * top-2), dmargin [k] (see orc_relaxed_choice) are optional. */
int orc_verify_block_pp(orc_state* s, int last, const int* draft, int k, int beta, double tau, int* pred, int* met,
                        real* margin, real* dmargin, real* logits_out, int* finished) {
  int V = s->m->cfg.vocab;
  int* tok = malloc(sizeof(int) * (size_t)k);
  real* lg = logits_out ? logits_out : malloc(sizeof(real) * (size_t)k * V);
  tok[0] = last;
  for (int i = 1; i < k; ++i) tok[i] = draft[i - 1] >= 0 ? draft[i - 1] : s->m->cfg.pad;
  int rc = orc_decode_block(s, tok, k, lg);
  if (rc == 0) {
    for (int i = 0; i < k; ++i)
      pred[i] = orc_relaxed_choice(lg + (size_t)i * V, V, draft[i], beta, tau, met ? &met[i] : NULL,
                                   margin ? &margin[i] : NULL, dmargin ? &dmargin[i] : NULL);
    rc = orc_accept(pred, draft, k, s->m->cfg.eos, finished);
  }
  free(tok);
  if (!logits_out) free(lg);
  return rc;
}

void orc_commit(orc_state* s, int n) { s->len += n; if (s->len < 0) s->len = 0; }

/* ------------------------------------------------------------------------------------------ */
/* Decoding loops                                                                             */
/* ------------------------------------------------------------------------------------------ */

/* Greedy autoregressive decoding: o_{j+1} = argmax P(. | o_<=j, x), until [EOS] or max_len tokens.
 * out [max_len], margin [max_len] optional.  Returns the number of tokens (an [EOS] is included). */
int orc_greedy(orc_state* s, int max_len, int* out, real* margin) {
  const orc_cfg* c = &s->m->cfg;
  real* lg = malloc(sizeof(real) * (size_t)c->vocab);
  int last = c->bos, n = 0;
  s->len = 0;
  while (n < max_len) {
    if (orc_decode_block(s, &last, 1, lg) != 0) break;
    int id; real v1, v2;
    orc_top2(lg, c->vocab, &id, &v1, NULL, &v2);
    if (margin) margin[n] = v1 - v2;
    out[n++] = id;
    s->len += 1;
    last = id;
    if (id == c->eos) break;
  }
  free(lg);
  return n;
}

/* Trace of a draft-verify run, filled when the pointers are non-null (capacity: max_len entries
 * each, since every iteration accepts at least one token). */
typedef struct {
  int* it_k;      /* block size offered per iteration */
  int* it_n;      /* tokens accepted per iteration */
  int iterations;
  long offered;   /* sum of k */
} orc_trace;

/* Draft-verify with a position-aligned draft stream: at accepted length len the block is
 * stream[len .. len+k), k = min(kmax, max_len - len).  This is the Verify substep of Section 3.2
 * with the drafts supplied from outside. */
int orc_draft_verify_stream(orc_state* s, const int* stream, int kmax, int max_len, int* out, orc_trace* tr) {
  const orc_cfg* c = &s->m->cfg;
  int* pred = malloc(sizeof(int) * (size_t)kmax);
  int last = c->bos, fin = 0;
  s->len = 0;
  if (tr) { tr->iterations = 0; tr->offered = 0; }
  while (!fin && s->len < max_len) {
    int k = kmax < max_len - s->len ? kmax : max_len - s->len;
    int n = orc_verify_block(s, last, stream + s->len, k, pred, NULL, NULL, &fin);
    if (n < 1) break;
    for (int i = 0; i < n; ++i) out[s->len + i] = pred[i];
    if (tr) {
      if (tr->it_k) tr->it_k[tr->iterations] = k;
      if (tr->it_n) tr->it_n[tr->iterations] = n;
      tr->iterations++; tr->offered += k;
    }
    last = pred[n - 1];
    s->len += n;
  }
  free(pred);
  return s->len;
}

/* Algorithm 1.  src[0..n_src-1] are x_1..x_n.  Internally x = (BOS, x_1..x_n, PAD).  When the suffix of
 * the output has a unique match ending at x_i, the block is x_{i+1..n} followed by the [PAD] slot,
 * which can never equal a prediction and so guarantees a bifurcation; otherwise one plain step
 * (a block of one sentinel slot).  Blocks are clipped to kmax and to the remaining length. */
int orc_iad(orc_state* s, const int* src, int n_src, int kmax, int max_len, int* out, orc_trace* tr) {
  const orc_cfg* c = &s->m->cfg;
  int* x = malloc(sizeof(int) * (size_t)(n_src + 2));
  int* o = malloc(sizeof(int) * (size_t)(max_len + 1));
  int* draft = malloc(sizeof(int) * (size_t)(n_src + 2));
  int* pred = malloc(sizeof(int) * (size_t)(n_src + 2));
  x[0] = c->bos;
  for (int i = 0; i < n_src; ++i) x[i + 1] = src[i];
  x[n_src + 1] = c->pad;
  o[0] = c->bos;
  int j = 0, fin = 0;
  s->len = 0;
  if (tr) { tr->iterations = 0; tr->offered = 0; }
  while (!fin && j < max_len) {
    int i = orc_suffix_match(o, j, x, n_src);
    int k = 1;
    draft[0] = -1;
    if (i >= 0) {
      k = 0;
      for (int t = i + 1; t <= n_src; ++t) draft[k++] = x[t];
      draft[k++] = -1;                       /* the [PAD] slot: compared, never equal */
    }
    if (k > kmax) { k = kmax; }
    if (k > max_len - j) k = max_len - j;
    int n = orc_verify_block(s, o[j], draft, k, pred, NULL, NULL, &fin);
    if (n < 1) break;
    for (int t = 0; t < n; ++t) { o[j + 1 + t] = pred[t]; out[j + t] = pred[t]; }
    if (tr) {
      if (tr->it_k) tr->it_k[tr->iterations] = k;
      if (tr->it_n) tr->it_n[tr->iterations] = n;
      tr->iterations++; tr->offered += k;
    }
    j += n;
    s->len = j;
  }
  free(x); free(o); free(draft); free(pred);
  return j;
}

/* Draft substep (Section 3.2, Section 3.2.1): the drafter's decoder reads (o_0..o_j, k x [MASK]) at
 * positions 0..j+k with bidirectional attention and no cache; drafts are the greedy choices at the k
 * mask positions.  prefix[0..j] includes BOS at index 0.  margin optional [k]. */
void orc_nar_draft(const orc_model* nar, const real* nar_mem, int S, const int* prefix, int j, int k,
                   int* draft, real* margin) {
  int T = j + 1 + k, V = nar->cfg.vocab;
  int* tok = malloc(sizeof(int) * (size_t)T);
  real* lg = malloc(sizeof(real) * (size_t)T * V);
  for (int t = 0; t <= j; ++t) tok[t] = prefix[t];
  for (int t = 0; t < k; ++t) tok[j + 1 + t] = nar->cfg.mask;
  orc_decode_full(nar, nar_mem, S, tok, T, 0, lg);
  for (int t = 0; t < k; ++t) {
    real v1, v2;
    orc_top2(lg + (size_t)(j + 1 + t) * V, V, &draft[t], &v1, NULL, &v2);
    if (margin) margin[t] = v1 - v2;
  }
  free(tok); free(lg);
}

/* Generalized mode loop (Section 3.2): Draft with the drafter, Verify with the AR model, accept up to
 * and including the bifurcation, until [EOS] or max_len.  If override != NULL the drafter still runs
 * but its block is replaced by override[len .. len+k) (used to impose an agreement rate when the
 * weights are random).  nar / nar_mem may be NULL only if override is given. */
int orc_gad(orc_state* s, const orc_model* nar, const real* nar_mem, const int* override, int kmax,
            int max_len, int* out, orc_trace* tr) {
  const orc_cfg* c = &s->m->cfg;
  int* o = malloc(sizeof(int) * (size_t)(max_len + 1));
  int* draft = malloc(sizeof(int) * (size_t)kmax);
  int* pred = malloc(sizeof(int) * (size_t)kmax);
  o[0] = c->bos;
  int j = 0, fin = 0;
  s->len = 0;
  if (tr) { tr->iterations = 0; tr->offered = 0; }
  while (!fin && j < max_len) {
    int k = kmax < max_len - j ? kmax : max_len - j;
    if (nar) orc_nar_draft(nar, nar_mem, s->S, o, j, k, draft, NULL);
    if (override) for (int t = 0; t < k; ++t) draft[t] = override[j + t];
    int n = orc_verify_block(s, o[j], draft, k, pred, NULL, NULL, &fin);
    if (n < 1) break;
    for (int t = 0; t < n; ++t) { o[j + 1 + t] = pred[t]; out[j + t] = pred[t]; }
    if (tr) {
      if (tr->it_k) tr->it_k[tr->iterations] = k;
      if (tr->it_n) tr->it_n[tr->iterations] = n;
      tr->iterations++; tr->offered += k;
    }
    j += n;
    s->len = j;
  }
  free(o); free(draft); free(pred);
  return j;
}

/* Generalized mode with the relaxed verification (Section 3.2.3): the loop of orc_gad with
 * orc_verify_block_pp in place of the exact-match verification. */
int orc_gad_pp(orc_state* s, const orc_model* nar, const real* nar_mem, const int* override, int kmax,
               int max_len, int beta, double tau, int* out, orc_trace* tr) {
  const orc_cfg* c = &s->m->cfg;
  int* o = malloc(sizeof(int) * (size_t)(max_len + 1));
  int* draft = malloc(sizeof(int) * (size_t)kmax);
  int* pred = malloc(sizeof(int) * (size_t)kmax);
  o[0] = c->bos;
  int j = 0, fin = 0;
  s->len = 0;
  if (tr) { tr->iterations = 0; tr->offered = 0; }
  while (!fin && j < max_len) {
    int k = kmax < max_len - j ? kmax : max_len - j;
    if (nar) orc_nar_draft(nar, nar_mem, s->S, o, j, k, draft, NULL);
    if (override) for (int t = 0; t < k; ++t) draft[t] = override[j + t];
    int n = orc_verify_block_pp(s, o[j], draft, k, beta, tau, pred, NULL, NULL, NULL, NULL, &fin);
    if (n < 1) break;
    for (int t = 0; t < n; ++t) { o[j + 1 + t] = pred[t]; out[j + t] = pred[t]; }
    if (tr) {
      if (tr->it_k) tr->it_k[tr->iterations] = k;
      if (tr->it_n) tr->it_n[tr->iterations] = n;
      tr->iterations++; tr->offered += k;
    }
    j += n;
    s->len = j;
  }
  free(o); free(draft); free(pred);
  return j;
}

int orc_real_size(void) { return (int)sizeof(real); }
