/*
 * hs_oracle.c -- CPU oracle for the shared-stage transformer step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against; nothing on the product path may call it.  It
 * shares no code, header, table or helper with the CUDA sources.
 *
 * What is computed: one batched step of an autoregressive transformer stage
 * (the "shared stage" of the paper, Sec. 2.2; "prefill builds the KV cache,
 * decode re-reads weights and the accumulated KV cache", Sec. 2.1) over a
 * mixed batch of chunked-prefill and decode sequences with a paged bf16 KV
 * cache.  The paper keeps the model execution of its runtime unchanged
 * (Sec. 5) and prints no formula for it, so the arithmetic below is the
 * textbook pre-norm decoder layer:
 *
 *   h   = rmsnorm(x; g_attn)            r = 1/sqrt(mean(x^2) + eps)
 *   q,k,v = h W_q^T + b_q, h W_k^T + b_k, h W_v^T + b_v   (weights are [out, in]; the biases are optional and
 *           added before RoPE, as in the checkpoints of the 7B-class backbones that carry them)
 *   q,k <- rope(q,k; position)          rotate-half pairs (i, i + Dh/2)
 *   cache[page(p)][slot(p)] <- bf16(k), bf16(v)     (all tokens first)
 *   o   = softmax(q K^T / sqrt(Dh)) V   keys 0..p read back from the cache
 *   x  += o W_o^T
 *   h2  = rmsnorm(x; g_mlp)
 *   x  += (silu(h2 W_g^T) * (h2 W_u^T)) W_d^T
 *
 * Arithmetic type: `real` (float by default; build with -DHSO_REAL=double for
 * the float64 variant used to bound the float32 rounding of this file).  The
 * only bf16 rounding is the KV cache write, which is interface-visible storage.
 *
 * Parity status: the paper prints no worked numeric example of the step, so
 * paper-level parity is unpinned.  Definition-level parity is pinned by the
 * CPU tests: softmax rows sum to 1, constant-V attention returns V, causal
 * brute force on tiny inputs, chunked prefill == full prefill, decode ==
 * last row of prefill, RoPE norm preservation and relative-position
 * property, paging permutation invariance, and a float64 cross-check against
 * library routines for the non-paged single-sequence case.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef HSO_REAL
#define HSO_REAL float
#endif
typedef HSO_REAL real;

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
  int32_t page_size, num_pages;
  float rms_eps, rope_base;
  int32_t bidirectional; /* 0: causal (a token sees the keys up to its own position); 1: every token of a
                          * sequence sees all of the sequence's keys, the cached ones and all new ones (the
                          * attention of a denoising / DiT-style block: no mask) */
} hso_config_t;

typedef struct {
  const real *g_attn, *w_q, *w_k, *w_v, *w_o, *g_mlp, *w_gate, *w_up, *w_down;
  const real *b_q, *b_k, *b_v; /* [Hq Dh], [Hkv Dh], [Hkv Dh]; NULL = no bias */
  /* Per-sequence modulation of a conditioned (DiT-style, "adaLN-Zero") block, [n_seqs][6][d], NULL = none:
   * rows 0..5 of sequence s are shift_a, scale_a, gate_a, shift_m, scale_m, gate_m and
   *   h_a = rmsnorm(x) g_attn (1 + scale_a) + shift_a,   x += gate_a * (attention output W_o^T),
   *   h_m = rmsnorm(x) g_mlp  (1 + scale_m) + shift_m,   x += gate_m * (MLP output),
   * all products element-wise over the d_model axis. */
  const real *mod;
} hso_layer_t;

/* Diagnostic switch (never the pass/fail oracle): bit mask of intermediates
 * that are rounded the way a 16-bit-operand tensor-core path would.
 * 1: h (both norms)  2: q  4: softmax weights P  8: o  16: act
 * 32: round h, o and act to fp16 (clamped to +-65504) instead of bf16 */
static int g_round_mask = 0;
void hso_set_operand_rounding(int mask) { g_round_mask = mask; }
int hso_sizeof_real(void) { return (int)sizeof(real); }

/* ---------------------------------------------------------------- bf16 -- */
/* Round-to-nearest-even float32 -> bfloat16 bits; inputs are finite. */
uint16_t hso_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}
float hso_bf16_to_float(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
static inline real round_bf16(real v) {
  return (real)hso_bf16_to_float(hso_bf16_rne((float)v));
}
static inline real round_f16(real v) {
  float f = (float)v;
  if (f > 65504.f) f = 65504.f;
  if (f < -65504.f) f = -65504.f;
  return (real)(float)(_Float16)f;
}
/* rounding of the activations that feed the projections (h, o, act) */
static inline real round_act(real v) { return (g_round_mask & 32) ? round_f16(v) : round_bf16(v); }

/* ------------------------------------------------------------- RMSNorm -- */
/* h[t,i] = x[t,i] * r_t * g[i],  r_t = 1/sqrt(mean_i x[t,i]^2 + eps). */
void hso_rmsnorm(int T, int d, const real *x, const real *g, float eps, real *h) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const real *xr = x + (size_t)t * d;
    real ss = 0;
    for (int i = 0; i < d; ++i) ss += xr[i] * xr[i];
    real r = (real)1 / (real)sqrt((double)(ss / (real)d + (real)eps));
    for (int i = 0; i < d; ++i) h[(size_t)t * d + i] = xr[i] * r * g[i];
  }
}

/* -------------------------------------------------------------- linear -- */
/* y[t,n] = sum_i a[t,i] * w[n,i]   (a: [T,K], w: [N,K], y: [T,N]).
 * The token loop is cut into groups of TB rows only so that one weight row
 * is reused from cache.  Every dot product is one i-loop over the whole K
 * range, but not a strictly sequential sum: the simd reduction lets the
 * compiler keep one partial sum per vector lane and add the lanes at the
 * end, so the order of the additions is the compiler's (a reassociation
 * of the same K terms; the float64 build bounds its effect at 1e-6). */
void hso_linear(int T, int N, int K, const real *a, const real *w, real *y) {
  enum { TB = 16 };
  int n_groups = (T + TB - 1) / TB;
#pragma omp parallel for schedule(dynamic, 1)
  for (int gidx = 0; gidx < n_groups; ++gidx) {
    int t0 = gidx * TB, t1 = t0 + TB < T ? t0 + TB : T;
    for (int n = 0; n < N; ++n) {
      const real *wr = w + (size_t)n * K;
      for (int t = t0; t < t1; ++t) {
        const real *ar = a + (size_t)t * K;
        real acc = 0;
#pragma omp simd reduction(+ : acc)
        for (int i = 0; i < K; ++i) acc += ar[i] * wr[i];
        y[(size_t)t * N + n] = acc;
      }
    }
  }
}

/* ---------------------------------------------------------------- RoPE -- */
/* Rotate-half RoPE on one token's heads z[n_heads][Dh] at absolute position
 * pos: theta_i = base^(-2i/Dh); the angle and its cos/sin are formed in
 * double and rounded to `real`. */
void hso_rope(int n_heads, int Dh, int pos, float base, real *z) {
  int half = Dh / 2;
  for (int i = 0; i < half; ++i) {
    double theta = pow((double)base, -2.0 * (double)i / (double)Dh);
    double phi = (double)pos * theta;
    real c = (real)cos(phi), s = (real)sin(phi);
    for (int h = 0; h < n_heads; ++h) {
      real *zh = z + (size_t)h * Dh;
      real a = zh[i], b = zh[i + half];
      zh[i] = a * c - b * s;
      zh[i + half] = b * c + a * s;
    }
  }
}

/* ---------------------------------------------------------------- SiLU -- */
real hso_silu(real z) { return z / ((real)1 + (real)exp(-(double)z)); }
float hso_silu_f32(float z) { return (float)hso_silu((real)z); }

/* ------------------------------------------------------------ KV cache -- */
/* Element offset of cache[layer][kv][page][kv_head][slot][0] (kv: 0 = K, 1 = V). */
static inline size_t kv_offset(const hso_config_t *c, int layer, int kv, int page, int hk, int slot) {
  size_t o = (size_t)layer * 2 + (size_t)kv;
  o = o * (size_t)c->num_pages + (size_t)page;
  o = o * (size_t)c->n_kv_heads + (size_t)hk;
  o = o * (size_t)c->page_size + (size_t)slot;
  return o * (size_t)c->head_dim;
}
size_t hso_kv_pool_elems(const hso_config_t *c) {
  return (size_t)c->n_layers * 2 * (size_t)c->num_pages * (size_t)c->n_kv_heads *
         (size_t)c->page_size * (size_t)c->head_dim;
}

/* ----------------------------------------------------------- attention -- */
/* One query vector q[Dh] (query head hq) at position pos attends keys
 * 0..pos of its sequence, read from the bf16 cache through the sequence's
 * block-table row.  probs (nullable) receives the pos+1 softmax weights. */
void hso_attend(const hso_config_t *c, const uint16_t *kv_pool, int layer, const int32_t *table_row,
                int pos, int hq, const real *q, real *o, real *probs) {
  int Dh = c->head_dim, G = c->n_q_heads / c->n_kv_heads, hk = hq / G, Pg = c->page_size;
  int n = pos + 1;
  real *s = (real *)malloc(sizeof(real) * (size_t)n);
  real scale = (real)1 / (real)sqrt((double)Dh);
  for (int j = 0; j < n; ++j) {
    const uint16_t *kr = kv_pool + kv_offset(c, layer, 0, table_row[j / Pg], hk, j % Pg);
    real acc = 0;
    for (int e = 0; e < Dh; ++e) acc += q[e] * (real)hso_bf16_to_float(kr[e]);
    s[j] = acc * scale;
  }
  real m = s[0];
  for (int j = 1; j < n; ++j) m = s[j] > m ? s[j] : m;
  real denom = 0;
  for (int j = 0; j < n; ++j) {
    s[j] = (real)exp((double)(s[j] - m));
    denom += s[j];
  }
  for (int e = 0; e < Dh; ++e) o[e] = 0;
  for (int j = 0; j < n; ++j) {
    const uint16_t *vr = kv_pool + kv_offset(c, layer, 1, table_row[j / Pg], hk, j % Pg);
    real wj = (g_round_mask & 4) ? round_bf16(s[j]) : s[j];
    for (int e = 0; e < Dh; ++e) o[e] += wj * (real)hso_bf16_to_float(vr[e]);
  }
  for (int e = 0; e < Dh; ++e) o[e] /= denom;
  if (probs)
    for (int j = 0; j < n; ++j) probs[j] = s[j] / denom;
  free(s);
}

/* ----------------------------------------------------------- one layer -- */
/* h[r, :] = h[r, :] * (1 + scale) + shift with the vectors of row r's sequence (mod == NULL: nothing).
 * seq_of[r] is the sequence of row r; `which` = 0 for the attention branch, 3 for the MLP branch. */
static void modulate(int R, int d, const real *mod, const int *seq_of, int which, real *h) {
  if (!mod) return;
  for (int r = 0; r < R; ++r) {
    const real *shift = mod + ((size_t)seq_of[r] * 6 + which) * d, *scale = shift + d;
    for (int i = 0; i < d; ++i) h[(size_t)r * d + i] = h[(size_t)r * d + i] * ((real)1 + scale[i]) + shift[i];
  }
}
/* x[r, :] += gate * t[r, :] (mod == NULL: gate = 1); `which` = 2 for the attention branch, 5 for the MLP. */
static void gated_add(int R, int d, const real *mod, const int *seq_of, int which, const real *t, real *x) {
  for (int r = 0; r < R; ++r) {
    const real *gate = mod ? mod + ((size_t)seq_of[r] * 6 + which) * d : NULL;
    for (int i = 0; i < d; ++i) x[(size_t)r * d + i] += (gate ? gate[i] : (real)1) * t[(size_t)r * d + i];
  }
}

/* y[t, :] += b for every row (b == NULL: nothing). */
static void add_bias(int T, int n, const real *b, real *y) {
  if (!b) return;
  for (int t = 0; t < T; ++t)
    for (int i = 0; i < n; ++i) y[(size_t)t * n + i] += b[i];
}

/*
 * Runs layer `layer` on the residual stream x[T,d] in place.
 *   q_len[s], ctx_len[s]: new / already cached tokens of sequence s; token j
 *   of its chunk has position ctx_len[s] + j.  block_tables[s*mpps + i] is the
 *   physical page of logical page i.
 *   row_mask (nullable, [T]): K/V of ALL tokens are always formed and written;
 *   everything after the cache write is evaluated only for rows with a
 *   non-zero mask, the other rows of x are left as they came in.
 *   kv_pre (nullable, [T][2][Hkv*Dh]): the k (after RoPE) and v values of this
 *   layer before their bf16 rounding.
 * Returns 0, or -1 on a malformed batch.
 */
int hso_layer(const hso_config_t *c, const hso_layer_t *w, int layer, uint16_t *kv_pool, int n_seqs,
              const int32_t *q_len, const int32_t *ctx_len, const int32_t *block_tables, int mpps,
              real *x, const uint8_t *row_mask, real *kv_pre) {
  int d = c->d_model, Hq = c->n_q_heads, Hkv = c->n_kv_heads, Dh = c->head_dim, F = c->d_ffn;
  int Pg = c->page_size;
  int T = 0;
  for (int s = 0; s < n_seqs; ++s) {
    if (q_len[s] < 1 || ctx_len[s] < 0) return -1;
    if ((ctx_len[s] + q_len[s] + Pg - 1) / Pg > mpps) return -1;
    T += q_len[s];
  }
  int *tok_seq = (int *)malloc(sizeof(int) * (size_t)T), *tok_pos = (int *)malloc(sizeof(int) * (size_t)T);
  for (int s = 0, t = 0; s < n_seqs; ++s)
    for (int j = 0; j < q_len[s]; ++j, ++t) {
      tok_seq[t] = s;
      tok_pos[t] = ctx_len[s] + j;
    }

  /* 1. attention norm */
  real *h = (real *)malloc(sizeof(real) * (size_t)T * d);
  hso_rmsnorm(T, d, x, w->g_attn, c->rms_eps, h);
  modulate(T, d, w->mod, tok_seq, 0, h);
  if (g_round_mask & 1)
    for (size_t i = 0; i < (size_t)T * d; ++i) h[i] = round_act(h[i]);

  /* 2. k, v of every token; RoPE on k; cache write (before any attention) */
  int KVd = Hkv * Dh;
  real *k = (real *)malloc(sizeof(real) * (size_t)T * KVd), *v = (real *)malloc(sizeof(real) * (size_t)T * KVd);
  hso_linear(T, KVd, d, h, w->w_k, k);
  hso_linear(T, KVd, d, h, w->w_v, v);
  add_bias(T, KVd, w->b_k, k);
  add_bias(T, KVd, w->b_v, v);
  for (int t = 0; t < T; ++t) {
    hso_rope(Hkv, Dh, tok_pos[t], c->rope_base, k + (size_t)t * KVd);
    if (kv_pre) {
      memcpy(kv_pre + ((size_t)t * 2 + 0) * KVd, k + (size_t)t * KVd, sizeof(real) * (size_t)KVd);
      memcpy(kv_pre + ((size_t)t * 2 + 1) * KVd, v + (size_t)t * KVd, sizeof(real) * (size_t)KVd);
    }
    int p = tok_pos[t], page = block_tables[(size_t)tok_seq[t] * mpps + p / Pg], slot = p % Pg;
    if (page < 0 || page >= c->num_pages) return -1;
    for (int hk = 0; hk < Hkv; ++hk) {
      uint16_t *kd = kv_pool + kv_offset(c, layer, 0, page, hk, slot);
      uint16_t *vd = kv_pool + kv_offset(c, layer, 1, page, hk, slot);
      for (int e = 0; e < Dh; ++e) {
        kd[e] = hso_bf16_rne((float)k[(size_t)t * KVd + hk * Dh + e]);
        vd[e] = hso_bf16_rne((float)v[(size_t)t * KVd + hk * Dh + e]);
      }
    }
  }
  free(k);
  free(v);

  /* rows evaluated past this point */
  int R = 0;
  int *rows = (int *)malloc(sizeof(int) * (size_t)T);
  for (int t = 0; t < T; ++t)
    if (!row_mask || row_mask[t]) rows[R++] = t;

  /* 3. q of the selected rows, RoPE */
  int Qd = Hq * Dh;
  real *hR = (real *)malloc(sizeof(real) * (size_t)R * d);
  for (int r = 0; r < R; ++r) memcpy(hR + (size_t)r * d, h + (size_t)rows[r] * d, sizeof(real) * (size_t)d);
  free(h);
  real *q = (real *)malloc(sizeof(real) * (size_t)R * Qd);
  hso_linear(R, Qd, d, hR, w->w_q, q);
  add_bias(R, Qd, w->b_q, q);
  for (int r = 0; r < R; ++r) hso_rope(Hq, Dh, tok_pos[rows[r]], c->rope_base, q + (size_t)r * Qd);
  if (g_round_mask & 2)
    for (size_t i = 0; i < (size_t)R * Qd; ++i) q[i] = round_bf16(q[i]);

  /* 4. causal GQA attention over the cache */
  real *o = (real *)malloc(sizeof(real) * (size_t)R * Qd);
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
  for (int r = 0; r < R; ++r)
    for (int hq = 0; hq < Hq; ++hq) {
      int t = rows[r];
      int last = c->bidirectional ? ctx_len[tok_seq[t]] + q_len[tok_seq[t]] - 1 : tok_pos[t];
      hso_attend(c, kv_pool, layer, block_tables + (size_t)tok_seq[t] * mpps, last, hq,
                 q + (size_t)r * Qd + (size_t)hq * Dh, o + (size_t)r * Qd + (size_t)hq * Dh, NULL);
    }
  free(q);
  if (g_round_mask & 8)
    for (size_t i = 0; i < (size_t)R * Qd; ++i) o[i] = round_act(o[i]);

  /* 5. output projection + residual */
  real *xR = (real *)malloc(sizeof(real) * (size_t)R * d), *tmp = (real *)malloc(sizeof(real) * (size_t)R * d);
  for (int r = 0; r < R; ++r) memcpy(xR + (size_t)r * d, x + (size_t)rows[r] * d, sizeof(real) * (size_t)d);
  hso_linear(R, d, Qd, o, w->w_o, tmp);
  int *seqR = (int *)malloc(sizeof(int) * (size_t)(R > 0 ? R : 1));
  for (int r = 0; r < R; ++r) seqR[r] = tok_seq[rows[r]];
  gated_add(R, d, w->mod, seqR, 2, tmp, xR);
  free(o);

  /* 6. MLP norm, SwiGLU */
  hso_rmsnorm(R, d, xR, w->g_mlp, c->rms_eps, hR);
  modulate(R, d, w->mod, seqR, 3, hR);
  if (g_round_mask & 1)
    for (size_t i = 0; i < (size_t)R * d; ++i) hR[i] = round_act(hR[i]);
  real *gate = (real *)malloc(sizeof(real) * (size_t)R * F), *up = (real *)malloc(sizeof(real) * (size_t)R * F);
  hso_linear(R, F, d, hR, w->w_gate, gate);
  hso_linear(R, F, d, hR, w->w_up, up);
  for (size_t i = 0; i < (size_t)R * F; ++i) {
    gate[i] = hso_silu(gate[i]) * up[i];
    if (g_round_mask & 16) gate[i] = round_act(gate[i]);
  }
  free(up);
  free(hR);

  /* 7. down projection + residual */
  hso_linear(R, d, F, gate, w->w_down, tmp);
  gated_add(R, d, w->mod, seqR, 5, tmp, xR);
  free(seqR);
  free(gate);
  free(tmp);
  for (int r = 0; r < R; ++r) memcpy(x + (size_t)rows[r] * d, xR + (size_t)r * d, sizeof(real) * (size_t)d);
  free(xR);
  free(rows);
  free(tok_seq);
  free(tok_pos);
  return 0;
}

/* ------------------------------------------------------------ the step -- */
/* y = residual stream after all layers, x_in[T,d] the step's input hidden
 * states.  row_mask (nullable) applies to the LAST layer only. */
int hso_step(const hso_config_t *c, const hso_layer_t *layers, uint16_t *kv_pool, int n_seqs,
             const int32_t *q_len, const int32_t *ctx_len, const int32_t *block_tables, int mpps,
             const real *x_in, real *y_out, const uint8_t *last_layer_row_mask) {
  int T = 0;
  for (int s = 0; s < n_seqs; ++s) T += q_len[s];
  memcpy(y_out, x_in, sizeof(real) * (size_t)T * c->d_model);
  for (int l = 0; l < c->n_layers; ++l) {
    int rc = hso_layer(c, layers + l, l, kv_pool, n_seqs, q_len, ctx_len, block_tables, mpps, y_out,
                       l == c->n_layers - 1 ? last_layer_row_mask : NULL, NULL);
    if (rc) return rc;
  }
  return 0;
}
