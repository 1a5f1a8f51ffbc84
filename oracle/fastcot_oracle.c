/*
 * CPU oracle for the Jacobi-window decode step (FastCoT, arXiv 2311.08263).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA library is
 * checked against.  It shares no code with the CUDA path, and only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may build or call it.
 *
 * What it computes
 *   - decoder forward: a Llama-style causal decoder (RMSNorm, rotary embedding with
 *     half-split pairing, grouped-query attention, SwiGLU FFN, untied LM head), the model
 *     family the paper evaluates (Experiment Settings).  fp32 arithmetic throughout.  For a bf16 model the K and V
 *     rows are rounded to bfloat16 where they are stored (the model's K/V tensors have the model dtype).
 *   - greedy autoregressive decoding: Eq. 1.
 *   - one Jacobi-window iteration: exact token + approximate tokens in one causal forward
 *     (Eq. 2-4), verification of the previous guesses one by one (Eq. 5), and the buffer /
 *     index update (Method, "Cache Update"; "Approximate Tokens Buffer" for its initialisation).
 *   - the hand-off of the approximate rationale: exact tokens + current approximate tokens +
 *     answer trigger, then greedy decoding of the answer (Method, "Overview of FastCoT" and
 *     "Trigger Answer"), and the iteration cap of "Iteration Stop Condition" (condition 1).
 *
 * Every output row is evaluated by the same scalar routine with a fixed summation order,
 * so row j of a window forward is bitwise the autoregressive forward of the same context.
 * That makes the paper's losslessness statement ("Overview of FastCoT": each forward yields at least
 * one token identical to autoregressive decoding) checkable exactly.
 *
 * Pins (tests/test_oracle_*.py): stream == greedy AR stream; closed form of the accept
 * count given the AR stream; brute force over all windows on tiny vocabularies; zero-matrix
 * closed form (stream = iterated permutation); attention/RoPE/RMSNorm special cases; an
 * independent fp64 library forward.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC (no -ffast-math: summation order is part of the spec).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t wdtype;            /* 0: weights are float32; 1: weights are bfloat16 bit patterns */
  float rms_eps, rope_theta, bias_beta;
  int32_t max_seq;           /* capacity of the K/V cache in tokens (committed + window) */
  int32_t kv_bf16;           /* 1: K and V are rounded to bfloat16 where they are stored (a bf16 model's K/V
                              * tensors are bf16); all arithmetic stays fp32.  0: K/V kept in fp32 */
} orc_shape;

typedef struct {             /* host pointers, row-major [out_features, in_features] */
  const void *tok_emb;
  const void *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *w_gate, *const *w_up, *const *w_down;
  const void *const *g_attn, *const *g_ffn;
  const void *g_final, *lm_head;
  const int32_t *bias_perm;  /* f: [vocab] or NULL */
} orc_weights;

typedef struct orc {
  orc_shape s;
  orc_weights w;
  float *kcache, *vcache;    /* [layer][max_seq][n_kv_heads*head_dim] */
  int32_t kv_len;            /* tokens whose K/V is committed */
  /* Jacobi state ("Approximate Tokens Buffer"): window = pending exact token + guesses */
  int32_t *prompt; int32_t prompt_len;
  int32_t *window; int32_t c;
  int32_t n_gen; int32_t refill; int32_t pad_id;
  /* optional trace of intermediates of the most recent forward (layer 0 and final) */
  float *trace_q, *trace_attn, *trace_x_out;
} orc;

/* ------------------------------------------------------------------ element access */
static inline float bf16_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16; float f; memcpy(&f, &u, 4); return f;
}
/* round to nearest even onto the bfloat16 grid (NaN stays NaN) */
float orc_round_bf16(float f) {
  uint32_t u; memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return f;
  u += 0x7fffu + ((u >> 16) & 1u);
  u &= 0xffff0000u;
  memcpy(&f, &u, 4); return f;
}
static inline float wload(const void *p, int wdtype, size_t i) {
  return wdtype ? bf16_to_f32(((const uint16_t *)p)[i]) : ((const float *)p)[i];
}

/* dot(w_row, x) over n terms; 16 interleaved partial sums added in a fixed order. */
static float dot_row(const void *w, int wdtype, size_t row, int n, const float *x) {
  float acc[16];
  for (int j = 0; j < 16; ++j) acc[j] = 0.f;
  int k = 0;
  if (wdtype) {
    const uint16_t *wr = (const uint16_t *)w + row * (size_t)n;
    for (; k + 16 <= n; k += 16)
      for (int j = 0; j < 16; ++j) acc[j] += bf16_to_f32(wr[k + j]) * x[k + j];
    for (int j = 0; k < n; ++k, ++j) acc[j] += bf16_to_f32(wr[k]) * x[k];
  } else {
    const float *wr = (const float *)w + row * (size_t)n;
    for (; k + 16 <= n; k += 16)
      for (int j = 0; j < 16; ++j) acc[j] += wr[k + j] * x[k + j];
    for (int j = 0; k < n; ++k, ++j) acc[j] += wr[k] * x[k];
  }
  float s = 0.f;
  for (int j = 0; j < 16; ++j) s += acc[j];
  return s;
}

/* Y[r, o] = dot(W[o, :], X[r, :]) for r < rows; parallel over output features only. */
static void linear(const void *w, int wdtype, int out_f, int in_f,
                   const float *x, int rows, float *y) {
#pragma omp parallel for schedule(static)
  for (int o = 0; o < out_f; ++o)
    for (int r = 0; r < rows; ++r)
      y[(size_t)r * out_f + o] = dot_row(w, wdtype, (size_t)o, in_f, x + (size_t)r * in_f);
}

/* h = x / sqrt(mean(x^2) + eps) * g */
static void rmsnorm(const float *x, const void *g, int wdtype, int d, float eps, float *h) {
  float ss = 0.f;
  for (int i = 0; i < d; ++i) ss += x[i] * x[i];
  float inv = 1.0f / sqrtf(ss / (float)d + eps);
  for (int i = 0; i < d; ++i) h[i] = x[i] * inv * wload(g, wdtype, (size_t)i);
}

/* rotary embedding of one head at absolute position pos: pairs (i, i + hd/2),
 * angle pos * theta^(-2i/hd). */
static void rope(float *v, int hd, int pos, float theta) {
  int half = hd / 2;
  for (int i = 0; i < half; ++i) {
    float freq = powf(theta, -2.0f * (float)i / (float)hd);
    float ang = (float)pos * freq;
    float cs = cosf(ang), sn = sinf(ang);
    float a = v[i], b = v[i + half];
    v[i] = a * cs - b * sn;
    v[i + half] = a * sn + b * cs;
  }
}

/* ------------------------------------------------------------------ decoder forward
 * Forward `n` tokens at absolute positions kv_len .. kv_len+n-1 on top of the committed
 * cache.  K/V of the new rows are written at cache slots kv_len .. kv_len+n-1 (scratch until
 * committed).  Row j attends keys 0 .. kv_len+j: the cache plus the causal part of the
 * window (Method, "FastCoT Inference": lossless and Jacobi decoding share one forward
 * through the causal mask).  logits_out: [n, vocab] or NULL.  argmax_out: [n] or NULL;
 * ties go to the lowest token id, NaN never wins.  Returns 0, or -1 on capacity overflow. */
int orc_forward(orc *o, const int32_t *tokens, int n, float *logits_out, int32_t *argmax_out) {
  const orc_shape *s = &o->s;
  const int d = s->d_model, hq = s->n_heads, hkv = s->n_kv_heads, hd = s->head_dim;
  const int f = s->d_ffn, V = s->vocab, wd = s->wdtype;
  const int qd = hq * hd, kvd = hkv * hd, group = hq / hkv;
  const int L = o->kv_len;
  if (n <= 0 || L + n > s->max_seq) return -1;
  for (int r = 0; r < n; ++r) if (tokens[r] < 0 || tokens[r] >= V) return -2;

  float *x = malloc(sizeof(float) * (size_t)n * d);
  float *h = malloc(sizeof(float) * (size_t)n * d);
  float *q = malloc(sizeof(float) * (size_t)n * qd);
  float *kk = malloc(sizeof(float) * (size_t)n * kvd);
  float *vv = malloc(sizeof(float) * (size_t)n * kvd);
  float *att = malloc(sizeof(float) * (size_t)n * qd);
  float *proj = malloc(sizeof(float) * (size_t)n * d);
  float *gate = malloc(sizeof(float) * (size_t)n * f);
  float *up = malloc(sizeof(float) * (size_t)n * f);

  for (int r = 0; r < n; ++r)
    for (int i = 0; i < d; ++i)
      x[(size_t)r * d + i] = wload(o->w.tok_emb, wd, (size_t)tokens[r] * d + i);

  for (int l = 0; l < s->n_layers; ++l) {
    float *kc = o->kcache + (size_t)l * s->max_seq * kvd;
    float *vc = o->vcache + (size_t)l * s->max_seq * kvd;
    for (int r = 0; r < n; ++r)
      rmsnorm(x + (size_t)r * d, o->w.g_attn[l], wd, d, s->rms_eps, h + (size_t)r * d);
    linear(o->w.wq[l], wd, qd, d, h, n, q);
    linear(o->w.wk[l], wd, kvd, d, h, n, kk);
    linear(o->w.wv[l], wd, kvd, d, h, n, vv);
    for (int r = 0; r < n; ++r) {
      int pos = L + r;
      for (int hh = 0; hh < hq; ++hh) rope(q + (size_t)r * qd + hh * hd, hd, pos, s->rope_theta);
      for (int hh = 0; hh < hkv; ++hh) rope(kk + (size_t)r * kvd + hh * hd, hd, pos, s->rope_theta);
      if (s->kv_bf16)
        for (int i = 0; i < kvd; ++i) {
          kk[(size_t)r * kvd + i] = orc_round_bf16(kk[(size_t)r * kvd + i]);
          vv[(size_t)r * kvd + i] = orc_round_bf16(vv[(size_t)r * kvd + i]);
        }
      memcpy(kc + (size_t)pos * kvd, kk + (size_t)r * kvd, sizeof(float) * kvd);
      memcpy(vc + (size_t)pos * kvd, vv + (size_t)r * kvd, sizeof(float) * kvd);
    }
    if (l == 0 && o->trace_q) memcpy(o->trace_q, q, sizeof(float) * (size_t)n * qd);

    const float scale = 1.0f / sqrtf((float)hd);
#pragma omp parallel for collapse(2) schedule(static)
    for (int r = 0; r < n; ++r) {
      for (int hh = 0; hh < hq; ++hh) {
        const int nk = L + r + 1;               /* keys 0 .. L+r */
        const int kvh = hh / group;
        const float *qv = q + (size_t)r * qd + hh * hd;
        float *sc = malloc(sizeof(float) * (size_t)nk);
        float mx = -INFINITY;
        for (int t = 0; t < nk; ++t) {
          const float *kt = kc + (size_t)t * kvd + kvh * hd;
          float a = 0.f;
          for (int i = 0; i < hd; ++i) a += qv[i] * kt[i];
          sc[t] = a * scale;
          if (sc[t] > mx) mx = sc[t];
        }
        float den = 0.f;
        for (int t = 0; t < nk; ++t) { sc[t] = expf(sc[t] - mx); den += sc[t]; }
        float *out = att + (size_t)r * qd + hh * hd;
        for (int i = 0; i < hd; ++i) out[i] = 0.f;
        for (int t = 0; t < nk; ++t) {
          const float p = sc[t] / den;
          const float *vt = vc + (size_t)t * kvd + kvh * hd;
          for (int i = 0; i < hd; ++i) out[i] += p * vt[i];
        }
        free(sc);
      }
    }
    if (l == 0 && o->trace_attn) memcpy(o->trace_attn, att, sizeof(float) * (size_t)n * qd);

    linear(o->w.wo[l], wd, d, qd, att, n, proj);
    for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += proj[i];

    for (int r = 0; r < n; ++r)
      rmsnorm(x + (size_t)r * d, o->w.g_ffn[l], wd, d, s->rms_eps, h + (size_t)r * d);
    linear(o->w.w_gate[l], wd, f, d, h, n, gate);
    linear(o->w.w_up[l], wd, f, d, h, n, up);
    for (size_t i = 0; i < (size_t)n * f; ++i) {
      float g = gate[i];
      gate[i] = (g / (1.0f + expf(-g))) * up[i];   /* silu(g) * u */
    }
    linear(o->w.w_down[l], wd, d, f, gate, n, proj);
    for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += proj[i];
  }
  if (o->trace_x_out) memcpy(o->trace_x_out, x, sizeof(float) * (size_t)n * d);

  {
    float *lg = logits_out ? logits_out : malloc(sizeof(float) * (size_t)n * V);
    for (int r = 0; r < n; ++r)
      rmsnorm(x + (size_t)r * d, o->w.g_final, wd, d, s->rms_eps, h + (size_t)r * d);
    linear(o->w.lm_head, wd, V, d, h, n, lg);
    for (int r = 0; r < n; ++r) {
      float *row = lg + (size_t)r * V;
      /* synthetic-workload logit bonus on token f(input token of this row) */
      if (o->w.bias_perm && s->bias_beta != 0.f) row[o->w.bias_perm[tokens[r]]] += s->bias_beta;
      if (argmax_out) {
        int best = 0; float bv = -INFINITY;
        for (int t = 0; t < V; ++t) if (row[t] > bv) { bv = row[t]; best = t; }
        argmax_out[r] = best;
      }
    }
    if (!logits_out) free(lg);
  }
  free(x); free(h); free(q); free(kk); free(vv); free(att); free(proj); free(gate); free(up);
  return 0;
}

/* ------------------------------------------------------------------ lifetime */
orc *orc_new(const orc_shape *s, const orc_weights *w) {
  if (!s || !w || s->n_heads % s->n_kv_heads || s->head_dim % 2) return NULL;
  orc *o = calloc(1, sizeof(orc));
  o->s = *s; o->w = *w;
  size_t n = (size_t)s->n_layers * s->max_seq * s->n_kv_heads * s->head_dim;
  o->kcache = calloc(n, sizeof(float));
  o->vcache = calloc(n, sizeof(float));
  return o;
}
void orc_free(orc *o) {
  if (!o) return;
  free(o->kcache); free(o->vcache); free(o->prompt); free(o->window); free(o);
}
void orc_set_trace(orc *o, float *q, float *attn, float *x_out) {
  o->trace_q = q; o->trace_attn = attn; o->trace_x_out = x_out;
}
int32_t orc_kv_len(const orc *o) { return o->kv_len; }
int32_t orc_n_gen(const orc *o) { return o->n_gen; }
int orc_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
/* Raw cache access for the window-step sweep: overwrite the K and V of `len` tokens of one
 * layer ([len, n_kv_heads*head_dim] each) and set the committed length. */
int orc_set_kv(orc *o, int layer, const float *k, const float *v, int len) {
  const orc_shape *s = &o->s;
  size_t kvd = (size_t)s->n_kv_heads * s->head_dim;
  if (layer < 0 || layer >= s->n_layers || len < 0 || len > s->max_seq) return -1;
  memcpy(o->kcache + (size_t)layer * s->max_seq * kvd, k, sizeof(float) * len * kvd);
  memcpy(o->vcache + (size_t)layer * s->max_seq * kvd, v, sizeof(float) * len * kvd);
  o->kv_len = len;
  return 0;
}

/* ------------------------------------------------------------------ Jacobi-window decoding
 * State ("Approximate Tokens Buffer"): committed tokens T[0..N-1]; K/V cached for T[0..N-2]; window w[0..c-1]
 * with w[0] = T[N-1] (exact, K/V not cached yet) and w[j>=1] the guess for token N-1+j. */

/* Initial / replacement guess for generated index g (0-based among generated tokens):
 * the prompt's own ids, cycled ("Approximate Tokens Buffer": initialised from the question's token ids),
 * or a pad id (the alternative the paper mentions). */
static int32_t refill_token(const orc *o, int g) {
  return o->refill == 1 ? o->pad_id : o->prompt[g % o->prompt_len];
}

/* Cache K/V of prompt[0..P-2]; prompt[P-1] becomes the pending exact token w[0]. */
int orc_prefill(orc *o, const int32_t *prompt, int P, int c, int refill, int pad_id) {
  if (P < 1 || c < 1 || P - 1 + c > o->s.max_seq) return -1;
  free(o->prompt); free(o->window);
  o->prompt = malloc(sizeof(int32_t) * P); memcpy(o->prompt, prompt, sizeof(int32_t) * P);
  o->prompt_len = P; o->c = c; o->refill = refill; o->pad_id = pad_id;
  o->window = malloc(sizeof(int32_t) * c);
  o->kv_len = 0; o->n_gen = 0;
  for (int start = 0; start < P - 1; start += 64) {       /* chunked only to bound scratch */
    int n = P - 1 - start < 64 ? P - 1 - start : 64;
    int rc = orc_forward(o, prompt + start, n, NULL, NULL);
    if (rc) return rc;
    o->kv_len += n;
  }
  o->window[0] = prompt[P - 1];
  for (int j = 1; j < c; ++j) o->window[j] = refill_token(o, j - 1);
  return 0;
}

/* Verification (Eq. 5) and buffer update (Method, "Cache Update") on plain arrays.
 * w[0..c-1]: the window that was fed (w[0] exact); a[j]: greedy token following window slot j;
 * n_gen: tokens generated before this step.  a[0] is always exact; a[j] is exact as long as every
 * guess w[1..j] equalled the exact token before it: check one by one.  Outputs: *k in [1, c],
 * accepted[0..k-1], and the new window: pending exact token a[k-1], then the still-unverified
 * outputs a[k..c-1] as the next guesses, then fresh guesses for the k-1 positions that no forward
 * has predicted yet (refill 0: prompt ids cycled by generated index; 1: pad_id). */
void orc_accept(const int32_t *w, const int32_t *a, int c, int n_gen, const int32_t *prompt, int P,
                int refill, int pad_id, int32_t *k_out, int32_t *accepted, int32_t *w_new) {
  int k = 1;
  while (k < c && w[k] == a[k - 1]) ++k;
  for (int j = 0; j < k; ++j) accepted[j] = a[j];
  *k_out = k;
  const int n1 = n_gen + k;
  w_new[0] = a[k - 1];
  for (int j = 1; j < c; ++j) {
    if (j <= c - k) w_new[j] = a[k - 1 + j];
    else w_new[j] = refill == 1 ? pad_id : prompt[(n1 + j - 1) % P];
  }
}

/* y[r, o] += dot(W[o, :], x[r, :]): the projection every GEMM of the step computes. */
void orc_linear_add(const void *w, int wdtype, int out_f, int in_f, const float *x, int rows, float *y) {
  float *t = malloc(sizeof(float) * (size_t)rows * out_f);
  linear(w, wdtype, out_f, in_f, x, rows, t);
  for (size_t i = 0; i < (size_t)rows * out_f; ++i) y[i] += t[i];
  free(t);
}

/* One iteration (Eq. 4, Eq. 5, cache update).  window_in (or NULL = keep the internal window)
 * must carry the pending exact token in slot 0; slots 1.. are free guesses.
 * Outputs: *accepted = k in [1, c]; accepted_tokens[0..k-1]; window_out[0..c-1] (the refreshed
 * window, also kept internally); logits_out (optional) [c, vocab]. */
int orc_jacobi_step(orc *o, const int32_t *window_in, int32_t *accepted, int32_t *accepted_tokens,
                    int32_t *window_out, float *logits_out) {
  const int c = o->c;
  if (!o->window) return -3;
  if (window_in) {
    if (window_in[0] != o->window[0]) return -4;
    memcpy(o->window, window_in, sizeof(int32_t) * c);
  }
  int32_t *a = malloc(sizeof(int32_t) * c);
  int rc = orc_forward(o, o->window, c, logits_out, a);
  if (rc) { free(a); return rc; }
  int32_t *w2 = malloc(sizeof(int32_t) * c);
  int32_t k;
  orc_accept(o->window, a, c, o->n_gen, o->prompt, o->prompt_len, o->refill, o->pad_id, &k,
             accepted_tokens, w2);
  *accepted = k;
  o->kv_len += k;                 /* K/V of rows 0..k-1 are already in place */
  o->n_gen += k;
  memcpy(o->window, w2, sizeof(int32_t) * c);
  if (window_out) memcpy(window_out, w2, sizeof(int32_t) * c);
  free(a); free(w2);
  return 0;
}

/* Change the number of rows per forward between iterations (the paper studies the context-window
 * length as a free parameter, "Context Window Length"; nothing in Eq. 4-5 ties one iteration's c to the
 * next).  The pending exact token stays in slot 0; guesses that still fit are kept; new slots get the
 * refill rule's guess for their generated index. */
int orc_set_window(orc *o, int c_new) {
  if (!o->window || c_new < 1 || o->kv_len + c_new > o->s.max_seq) return -1;
  int32_t *w2 = malloc(sizeof(int32_t) * c_new);
  for (int j = 0; j < c_new; ++j)
    w2[j] = j < o->c ? o->window[j] : refill_token(o, o->n_gen + j - 1);
  free(o->window);
  o->window = w2; o->c = c_new;
  return 0;
}

/* Iterate until max_tokens are committed, eos_id is committed (eos_id < 0: never) or max_iters forwards
 * have run (max_iters <= 0: no cap; "Iteration Stop Condition": an upper bound on the iterations, and a
 * verified EOS).  The stream is cut at max_tokens and just after the first EOS; accept_counts[i]
 * (optional, up to max_tokens entries) gets the per-step count after that cut.  Returns the stream length. */
int orc_generate(orc *o, int max_tokens, int eos_id, int max_iters, int32_t *out_tokens,
                 int32_t *accept_counts, int32_t *n_steps) {
  int n = 0, steps = 0, done = 0;
  int32_t *acc = malloc(sizeof(int32_t) * o->c);
  while (n < max_tokens && !done && (max_iters <= 0 || steps < max_iters)) {
    int32_t k;
    int rc = orc_jacobi_step(o, NULL, &k, acc, NULL, NULL);
    if (rc) { free(acc); return rc; }
    int kept = 0;
    for (int j = 0; j < k && n < max_tokens && !done; ++j) {
      out_tokens[n++] = acc[j]; ++kept;
      if (eos_id >= 0 && acc[j] == eos_id) done = 1;
    }
    if (accept_counts) accept_counts[steps] = kept;
    ++steps;
  }
  if (n_steps) *n_steps = steps;
  free(acc);
  return n;
}

/* Hand-off of the approximate rationale ("Overview of FastCoT", last step; "Trigger Answer"): when the
 * iteration stops, everything generated so far - the exact tokens AND the approximate tokens still in
 * the window - is joined with the answer trigger, and the answer is decoded greedily from there.
 * Context = committed cache | w[0] (pending exact) | w[1..c-1] (approximate, taken as they are) |
 * trigger[0..n_trig-1]; all of it is committed to the cache except its last token, which becomes the
 * pending token of a plain autoregressive decode (Eq. 1) of up to max_answer tokens (cut after eos_id).
 * Afterwards the Jacobi state is gone (the buffer was consumed): prefill again before iterating.
 * Returns the number of answer tokens. */
int orc_finish_with_trigger(orc *o, const int32_t *trigger, int n_trig, int max_answer, int eos_id,
                            int32_t *answer) {
  if (!o->window || n_trig < 0 || max_answer < 0) return -1;
  const int n_ctx = o->c + n_trig;                 /* rows: window then trigger */
  if (o->kv_len + n_ctx + max_answer > o->s.max_seq) return -1;
  int32_t *ctx = malloc(sizeof(int32_t) * n_ctx);
  memcpy(ctx, o->window, sizeof(int32_t) * o->c);
  for (int j = 0; j < n_trig; ++j) ctx[o->c + j] = trigger[j];
  for (int j = 0; j < n_ctx; ++j) if (ctx[j] < 0 || ctx[j] >= o->s.vocab) { free(ctx); return -2; }
  for (int start = 0; start < n_ctx - 1; start += 64) {   /* chunked only to bound scratch */
    int n = n_ctx - 1 - start < 64 ? n_ctx - 1 - start : 64;
    int rc = orc_forward(o, ctx + start, n, NULL, NULL);
    if (rc) { free(ctx); return rc; }
    o->kv_len += n;
  }
  int32_t tok = ctx[n_ctx - 1];
  free(ctx);
  int n = 0;
  while (n < max_answer) {
    int32_t nxt;
    int rc = orc_forward(o, &tok, 1, NULL, &nxt);
    if (rc) return rc;
    o->kv_len += 1;
    answer[n++] = nxt;
    tok = nxt;
    if (eos_id >= 0 && nxt == eos_id) break;
  }
  free(o->window); o->window = NULL; o->c = 0;
  return n;
}

/* Plain greedy autoregressive decoding (Eq. 1) from the same prefill convention: one row per
 * forward, commit it, feed its argmax back. */
int orc_ar_generate(orc *o, const int32_t *prompt, int P, int max_tokens, int eos_id,
                    int32_t *out_tokens, float *margins /* optional [max_tokens] */) {
  int rc = orc_prefill(o, prompt, P, 1, 1, 0);
  if (rc) return rc;
  int32_t tok = prompt[P - 1];
  float *lg = malloc(sizeof(float) * o->s.vocab);
  int n = 0;
  while (n < max_tokens) {
    int32_t nxt;
    rc = orc_forward(o, &tok, 1, lg, &nxt);
    if (rc) { free(lg); return rc; }
    o->kv_len += 1;
    if (margins) {
      float second = -INFINITY;
      for (int t = 0; t < o->s.vocab; ++t) if (t != nxt && lg[t] > second) second = lg[t];
      margins[n] = lg[nxt] - second;
    }
    out_tokens[n++] = nxt;
    tok = nxt;
    if (eos_id >= 0 && nxt == eos_id) break;
  }
  free(lg);
  return n;
}

/* Copy out the first `len` cached tokens of one layer ([len, n_kv_heads*head_dim] each). */
int orc_get_kv(const orc *o, int layer, float *k, float *v, int len) {
  const orc_shape *s = &o->s;
  size_t kvd = (size_t)s->n_kv_heads * s->head_dim;
  if (layer < 0 || layer >= s->n_layers || len < 0 || len > s->max_seq) return -1;
  memcpy(k, o->kcache + (size_t)layer * s->max_seq * kvd, sizeof(float) * len * kvd);
  memcpy(v, o->vcache + (size_t)layer * s->max_seq * kvd, sizeof(float) * len * kvd);
  return 0;
}
