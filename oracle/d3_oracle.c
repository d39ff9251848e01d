/*
 * d3_oracle.c -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow CPU restatement of Position-Aware Depth Decay Decoding (D3):
 * the autoregressive decode of a Llama-style decoder in which generated token
 * T_i runs only floor(L * alpha^i) decoder blocks (Abstract; Sec. 3.4), the
 * skipped blocks being one contiguous window that begins at the "flex layer"
 * start id (Appendix, Table "HP description": drop-layer set), with the hidden
 * state carried unchanged through skipped blocks and their KV-cache entries
 * filled by copy / recompute / not at all (Sec. 1 (i); Sec. 3.2).
 *
 * Only the tests, the smoke check and the CPU-baseline timing may call this
 * file.  It shares no code, header, table or constant with the CUDA library
 * and neither includes the other.
 *
 * Arithmetic type: D3O_REAL (double unless overridden at compile time with
 * -DD3O_REAL=float).  Weights arrive as bf16 bit patterns (uint16) and are
 * widened exactly; every sum runs in index order, one accumulator, no
 * blocking, no fusion, no reordering.  OpenMP only splits independent output
 * elements across threads.
 *
 * Pins (tests marked "not gpu"):
 *   depth rule          closed form, the six average-layer figures printed in
 *                       the main-results table, monotonicity, nesting
 *   block / full model  the HuggingFace Llama implementation (the one the
 *                       paper patched) on the same weights, MHA and GQA
 *   truncated stacks    lm_head(norm(h^n)) of the library's hidden states
 *                       (TAIL anchor); the library model with the window's
 *                       layers deleted (START anchor)
 *   cache logic         cached decode == whole-sequence forward without cache
 *   fill modes          logits independent of the fill mode under a fixed
 *                       (alpha, start), skipped entries poisoned with NaN
 *   textbook properties softmax, RMSNorm, RoPE closed forms and invariants
 *   caller-given depths the step with depths = floor(L alpha^i) equals the alpha step
 *                       (itself pinned above); linear decay: end points, monotonicity
 *                       and the floor-sum identity sum_{i<n} floor(a i / n) =
 *                       ((a-1)(n-1) + gcd(a,n) - 1) / 2
 *   bf16 cache storage  round_bf16: hand-listed bit patterns (ties both ways, carry
 *                       into the exponent, subnormals, overflow, a value that
 *                       rounding twice would get wrong) and a sweep against
 *                       the library conversion of fp32 inputs
 * Parity unpinned: the VALUES that fill modes COPY / RECOMPUTE leave in the
 * cache when the caller raises alpha between steps (the paper never states
 * which rule D3 itself uses); only their own definitions below fix them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef D3O_REAL
#define D3O_REAL double
#endif
typedef D3O_REAL real;

enum { D3O_ANCHOR_START = 0, D3O_ANCHOR_TAIL = 1 };
enum { D3O_FILL_NONE = 0, D3O_FILL_COPY = 1, D3O_FILL_RECOMPUTE = 2 };

typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  double rms_eps, rope_base;
  int32_t max_slots, max_seq;
  int32_t start_id; /* first droppable layer, 0-based */
  int32_t anchor;
  int32_t kv_fill;
  int32_t kv_round_bf16; /* diagnostic: round K,V to bf16 when stored */
} d3o_config;

typedef struct {
  const uint16_t *embed;      /* [vocab][d] */
  const uint16_t *lm_head;    /* [vocab][d] */
  const uint16_t *final_norm; /* [d] */
  const uint16_t *const *attn_norm; /* L x [d] */
  const uint16_t *const *wq;        /* L x [Hq*dh][d] */
  const uint16_t *const *wk;        /* L x [Hkv*dh][d] */
  const uint16_t *const *wv;        /* L x [Hkv*dh][d] */
  const uint16_t *const *wo;        /* L x [d][Hq*dh] */
  const uint16_t *const *mlp_norm;  /* L x [d] */
  const uint16_t *const *w_gate;    /* L x [f][d] */
  const uint16_t *const *w_up;      /* L x [f][d] */
  const uint16_t *const *w_down;    /* L x [d][f] */
} d3o_weights;

typedef struct {
  d3o_config c;
  d3o_weights w;
  const uint16_t **ptrs; /* owned copy of the nine per-layer pointer arrays */
  real *K, *V;           /* [L][slot][max_seq][Hkv][dh] */
  int32_t *pos;          /* tokens in each slot's cache; -1 = never prefilled */
} d3o_model;

/* ------------------------------------------------------------------ helpers */

static real bf16_to_real(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (real)f;
}

/* The bf16 value nearest to x, ties to the even significand, returned widened:
 * ONE rounding of the value as it stands (a detour through fp32 would round
 * twice).  bf16 = 8 significand bits, exponent range of fp32: for |x| in
 * [2^e, 2^(e+1)) the spacing is 2^(e-7), below 2^-126 it stays 2^-133
 * (subnormals), and what rounds to 2^128 or beyond is infinity.  Zeros,
 * infinities and NaN pass through. */
static real round_bf16(real x) {
  double v = (double)x;
  if (v == 0.0 || isnan(v) || isinf(v)) return x;
  int e = ilogb(v);
  if (e < -126) e = -126;
  double quantum = ldexp(1.0, e - 7);
  double r = nearbyint(v / quantum) * quantum; /* default rounding mode: nearest, ties to even */
  if (fabs(r) >= ldexp(1.0, 128)) r = copysign(INFINITY, v);
  return (real)r;
}

/* test access to the storage rounding */
void d3o_round_bf16(const real *in, int32_t n, real *out) {
  for (int32_t k = 0; k < n; ++k) out[k] = round_bf16(in[k]);
}

static size_t kv_index(const d3o_config *c, int l, int slot, int t) {
  size_t per_tok = (size_t)c->n_kv_heads * c->head_dim;
  return ((((size_t)l * c->max_slots + slot) * c->max_seq) + t) * per_tok;
}

/* y[r] = sum_k W[r][k] a[k],  W row-major [rows][cols] */
static void matvec(const uint16_t *W, int rows, int cols, const real *a, real *y) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    const uint16_t *w = W + (size_t)r * cols;
    real s = 0;
    for (int k = 0; k < cols; ++k) s += bf16_to_real(w[k]) * a[k];
    y[r] = s;
  }
}

/* RMSNorm: x * 1/sqrt(mean(x^2) + eps), times the gain */
void d3o_rmsnorm(const real *x, const uint16_t *gain, int d, double eps, real *out) {
  real ss = 0;
  for (int k = 0; k < d; ++k) ss += x[k] * x[k];
  real inv = (real)1 / (real)sqrt((double)(ss / (real)d) + eps);
  for (int k = 0; k < d; ++k) out[k] = x[k] * inv * bf16_to_real(gain[k]);
}

/* Rotary embedding on one head vector, half-split pairing (j, j + dh/2),
 * theta_j = base^(-2j/dh); (a, b) -> (a cos - b sin, a sin + b cos). */
void d3o_rope(real *v, int dh, int pos, double base) {
  int half = dh / 2;
  for (int j = 0; j < half; ++j) {
    double theta = pow(base, -2.0 * (double)j / (double)dh);
    double ang = (double)pos * theta;
    real c = (real)cos(ang), s = (real)sin(ang);
    real a = v[j], b = v[j + half];
    v[j] = a * c - b * s;
    v[j + half] = a * s + b * c;
  }
}

/* softmax with the maximum subtracted */
void d3o_softmax(real *s, int n) {
  real mx = s[0];
  for (int t = 1; t < n; ++t)
    if (s[t] > mx) mx = s[t];
  real sum = 0;
  for (int t = 0; t < n; ++t) {
    s[t] = (real)exp((double)(s[t] - mx));
    sum += s[t];
  }
  for (int t = 0; t < n; ++t) s[t] /= sum;
}

static real silu(real z) { return z / ((real)1 + (real)exp((double)-z)); }

/* ------------------------------------------------------------ depth schedule */

/* floor(L * alpha^i): layers retained when generating T_i (Abstract; Sec. 3.4).
 * alpha^i by i sequential multiplications. */
int32_t d3o_depth(int32_t L, double alpha, int64_t i) {
  if (L < 0 || i < 0 || !(alpha > 0.0) || !(alpha <= 1.0)) return -1;
  double p = 1.0;
  for (int64_t t = 0; t < i; ++t) {
    p *= alpha;
    if (p * (double)L < 1.0) { /* floor stays 0 from here on */
      return 0;
    }
  }
  return (int32_t)floor((double)L * p);
}

/* the same value through the library power function */
int32_t d3o_depth_pow(int32_t L, double alpha, int64_t i) {
  if (L < 0 || i < 0 || !(alpha > 0.0) || !(alpha <= 1.0)) return -1;
  return (int32_t)floor((double)L * pow(alpha, (double)i));
}

/* Retained count n and dropped window [lo, hi) for token T_i.
 * START (the paper's rule, Appendix Table "HP description"): the window opens
 * at start_id and holds L - n layers, n never falling below start_id so that
 * the window ends at the last layer at the latest.
 * TAIL (the Early-Exit direction, Sec. 1 (ii)): the last L - n layers. */
static int32_t window_of_depth(int32_t L, int32_t n, int32_t start_id, int32_t anchor, int32_t *lo,
                               int32_t *hi);

int32_t d3o_window(int32_t L, double alpha, int64_t i, int32_t start_id, int32_t anchor,
                   int32_t *lo, int32_t *hi) {
  return window_of_depth(L, d3o_depth(L, alpha, i), start_id, anchor, lo, hi);
}

/* The same window for a retained count n given by the caller (any schedule). */
int32_t d3o_window_of_depth(int32_t L, int32_t n, int32_t start_id, int32_t anchor, int32_t *lo,
                            int32_t *hi) {
  if (n > L) return -1;
  return window_of_depth(L, n, start_id, anchor, lo, hi);
}

/* Linear decay between an upper and a lower bound of executed layers (the shape
 * the paper ascribes to SkipDecode, Sec. 3.4 and Sec. 4.1 "Comparison Methods";
 * its constants are not given there, so they are parameters): the count falls
 * from `upper` at i = 0 to `lower` at i = span in equal steps and stays there,
 *   n(i) = upper - floor((upper - lower) * min(i, span) / span). */
int32_t d3o_depth_linear(int32_t upper, int32_t lower, int64_t span, int64_t i) {
  if (upper < 0 || lower < 0 || lower > upper || span < 1 || i < 0) return -1;
  int64_t t = i < span ? i : span;
  int64_t drop = 0; /* floor(D * t / span) by counting: D * t = drop * span + rest */
  int64_t num = (int64_t)(upper - lower) * t;
  while ((drop + 1) * span <= num) ++drop;
  return (int32_t)(upper - drop);
}

static int32_t window_of_depth(int32_t L, int32_t n, int32_t start_id, int32_t anchor, int32_t *lo,
                               int32_t *hi) {
  if (n < 0 || start_id < 0 || start_id > L) return -1;
  if (anchor == D3O_ANCHOR_TAIL) {
    *lo = n;
    *hi = L;
    return n;
  }
  if (anchor != D3O_ANCHOR_START) return -1;
  if (n < start_id) n = start_id;
  *lo = start_id;
  *hi = start_id + (L - n);
  return n;
}

/* Batch schedule: per row retained count and window, the order of rows by
 * retained count descending (ties by caller row), and per layer the number of
 * rows that run it. */
int32_t d3o_schedule(int32_t L, double alpha, int32_t start_id, int32_t anchor, int32_t B,
                     const int32_t *gen_index, int32_t *n, int32_t *lo, int32_t *hi,
                     int32_t *perm, int32_t *m_per_layer, int64_t *rows_layers,
                     int32_t *layers_touched) {
  for (int b = 0; b < B; ++b) {
    n[b] = d3o_window(L, alpha, gen_index[b], start_id, anchor, &lo[b], &hi[b]);
    if (n[b] < 0) return -1;
  }
  for (int b = 0; b < B; ++b) perm[b] = b;
  for (int a = 1; a < B; ++a) { /* insertion sort: stable */
    int32_t v = perm[a];
    int j = a - 1;
    while (j >= 0 && n[perm[j]] < n[v]) {
      perm[j + 1] = perm[j];
      --j;
    }
    perm[j + 1] = v;
  }
  int64_t tot = 0;
  int32_t touched = 0;
  for (int l = 0; l < L; ++l) {
    int32_t m = 0;
    for (int b = 0; b < B; ++b)
      if (!(lo[b] <= l && l < hi[b])) ++m;
    m_per_layer[l] = m;
    tot += m;
    if (m > 0) ++touched;
  }
  *rows_layers = tot;
  *layers_touched = touched;
  return 0;
}

/* -------------------------------------------------------------------- model */

int d3o_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int d3o_real_bytes(void) { return (int)sizeof(real); }

d3o_model *d3o_create(const d3o_config *c, const d3o_weights *w) {
  if (!c || !w) return NULL;
  if (c->n_layers < 1 || c->d_model < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 ||
      c->head_dim < 2 || (c->head_dim & 1) || c->d_ffn < 1 || c->vocab < 1 ||
      c->n_q_heads % c->n_kv_heads != 0 || c->max_slots < 1 || c->max_seq < 1 ||
      c->start_id < 0 || c->start_id > c->n_layers)
    return NULL;
  d3o_model *m = (d3o_model *)calloc(1, sizeof(d3o_model));
  if (!m) return NULL;
  m->c = *c;
  m->w = *w;
  int L = c->n_layers;
  m->ptrs = (const uint16_t **)malloc(sizeof(void *) * 9 * (size_t)L);
  const uint16_t *const *src[9] = {w->attn_norm, w->wq, w->wk,     w->wv,  w->wo,
                                   w->mlp_norm,  w->w_gate, w->w_up, w->w_down};
  for (int a = 0; a < 9; ++a)
    for (int l = 0; l < L; ++l) m->ptrs[a * L + l] = src[a][l];
  m->w.attn_norm = m->ptrs + 0 * L;
  m->w.wq = m->ptrs + 1 * L;
  m->w.wk = m->ptrs + 2 * L;
  m->w.wv = m->ptrs + 3 * L;
  m->w.wo = m->ptrs + 4 * L;
  m->w.mlp_norm = m->ptrs + 5 * L;
  m->w.w_gate = m->ptrs + 6 * L;
  m->w.w_up = m->ptrs + 7 * L;
  m->w.w_down = m->ptrs + 8 * L;
  size_t kv = kv_index(c, L, 0, 0);
  m->K = (real *)calloc(kv, sizeof(real));
  m->V = (real *)calloc(kv, sizeof(real));
  m->pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)c->max_slots);
  if (!m->K || !m->V || !m->pos || !m->ptrs) return NULL;
  for (int s = 0; s < c->max_slots; ++s) m->pos[s] = -1;
  return m;
}

void d3o_destroy(d3o_model *m) {
  if (!m) return;
  free(m->K);
  free(m->V);
  free(m->pos);
  free((void *)m->ptrs);
  free(m);
}

/* every cache entry := NaN, so that reading an entry nobody wrote shows */
void d3o_poison_kv(d3o_model *m) {
  size_t kv = kv_index(&m->c, m->c.n_layers, 0, 0);
  for (size_t a = 0; a < kv; ++a) {
    m->K[a] = (real)NAN;
    m->V[a] = (real)NAN;
  }
}

void d3o_set_policy(d3o_model *m, int32_t start_id, int32_t anchor, int32_t kv_fill) {
  m->c.start_id = start_id;
  m->c.anchor = anchor;
  m->c.kv_fill = kv_fill;
}

int32_t d3o_slot_pos(const d3o_model *m, int32_t slot) {
  if (slot < 0 || slot >= m->c.max_slots) return -2;
  return m->pos[slot];
}

/* read one cache entry back (tests of the fill modes) */
void d3o_read_kv(const d3o_model *m, int32_t l, int32_t slot, int32_t t, double *k_out,
                 double *v_out) {
  size_t base = kv_index(&m->c, l, slot, t);
  int n = m->c.n_kv_heads * m->c.head_dim;
  for (int a = 0; a < n; ++a) {
    k_out[a] = (double)m->K[base + a];
    v_out[a] = (double)m->V[base + a];
  }
}

/* keys and values of layer l for the token at position pos, from hidden x */
static void project_kv(const d3o_model *m, int l, const real *x, int pos, real *a, real *k,
                       real *v) {
  const d3o_config *c = &m->c;
  int dh = c->head_dim, nkv = c->n_kv_heads * dh;
  d3o_rmsnorm(x, m->w.attn_norm[l], c->d_model, c->rms_eps, a);
  matvec(m->w.wk[l], nkv, c->d_model, a, k);
  matvec(m->w.wv[l], nkv, c->d_model, a, v);
  for (int h = 0; h < c->n_kv_heads; ++h) d3o_rope(k + h * dh, dh, pos, c->rope_base);
}

static void store_kv(d3o_model *m, int l, int slot, int pos, const real *k, const real *v) {
  const d3o_config *c = &m->c;
  size_t base = kv_index(c, l, slot, pos);
  int nkv = c->n_kv_heads * c->head_dim;
  for (int a = 0; a < nkv; ++a) {
    m->K[base + a] = c->kv_round_bf16 ? round_bf16(k[a]) : k[a];
    m->V[base + a] = c->kv_round_bf16 ? round_bf16(v[a]) : v[a];
  }
}

/* One Llama decoder block on the token at cache position pos of `slot`:
 * pre-norm attention over positions 0..pos (its own included) with grouped
 * KV heads, residual; pre-norm SwiGLU MLP, residual.  x is updated in place. */
static void block(d3o_model *m, int l, real *x, int slot, int pos) {
  const d3o_config *c = &m->c;
  int d = c->d_model, dh = c->head_dim, Hq = c->n_q_heads, Hkv = c->n_kv_heads;
  int nq = Hq * dh, nkv = Hkv * dh, f = c->d_ffn, group = Hq / Hkv;
  real *a = (real *)malloc(sizeof(real) * (size_t)d);
  real *q = (real *)malloc(sizeof(real) * (size_t)nq);
  real *k = (real *)malloc(sizeof(real) * (size_t)nkv);
  real *v = (real *)malloc(sizeof(real) * (size_t)nkv);
  real *o = (real *)malloc(sizeof(real) * (size_t)nq);
  real *y = (real *)malloc(sizeof(real) * (size_t)d);
  real *g = (real *)malloc(sizeof(real) * (size_t)f);
  real *u = (real *)malloc(sizeof(real) * (size_t)f);
  real *sc = (real *)malloc(sizeof(real) * (size_t)(pos + 1));

  project_kv(m, l, x, pos, a, k, v); /* leaves a = RMSNorm(x) */
  matvec(m->w.wq[l], nq, d, a, q);
  for (int h = 0; h < Hq; ++h) d3o_rope(q + h * dh, dh, pos, c->rope_base);
  store_kv(m, l, slot, pos, k, v);

  real scale = (real)1 / (real)sqrt((double)dh);
  for (int h = 0; h < Hq; ++h) {
    int kvh = h / group;
    for (int t = 0; t <= pos; ++t) {
      const real *kt = m->K + kv_index(c, l, slot, t) + (size_t)kvh * dh;
      real s = 0;
      for (int e = 0; e < dh; ++e) s += q[h * dh + e] * kt[e];
      sc[t] = s * scale;
    }
    d3o_softmax(sc, pos + 1);
    for (int e = 0; e < dh; ++e) {
      real s = 0;
      for (int t = 0; t <= pos; ++t)
        s += sc[t] * m->V[kv_index(c, l, slot, t) + (size_t)kvh * dh + e];
      o[h * dh + e] = s;
    }
  }
  matvec(m->w.wo[l], d, nq, o, y);
  for (int e = 0; e < d; ++e) x[e] += y[e];

  d3o_rmsnorm(x, m->w.mlp_norm[l], d, c->rms_eps, a);
  matvec(m->w.w_gate[l], f, d, a, g);
  matvec(m->w.w_up[l], f, d, a, u);
  for (int e = 0; e < f; ++e) u[e] = silu(g[e]) * u[e];
  matvec(m->w.w_down[l], d, f, u, y);
  for (int e = 0; e < d; ++e) x[e] += y[e];

  free(a); free(q); free(k); free(v); free(o); free(y); free(g); free(u); free(sc);
}

/* Missing KV of a skipped layer l for the token at `pos` (Sec. 3.2):
 * NONE leaves the entry alone; COPY takes the token's own K,V from the layer
 * just below the window (zeros when the window opens at layer 0); RECOMPUTE
 * projects the carried hidden state with layer l's own norm, W_k, W_v. */
static void fill_kv(d3o_model *m, int l, int slot, int pos, const real *x, int lo) {
  const d3o_config *c = &m->c;
  int nkv = c->n_kv_heads * c->head_dim;
  if (c->kv_fill == D3O_FILL_NONE) return;
  size_t dst = kv_index(c, l, slot, pos);
  if (c->kv_fill == D3O_FILL_COPY) {
    if (lo == 0) {
      for (int a = 0; a < nkv; ++a) m->K[dst + a] = m->V[dst + a] = 0;
    } else {
      size_t src = kv_index(c, lo - 1, slot, pos);
      for (int a = 0; a < nkv; ++a) {
        m->K[dst + a] = m->K[src + a];
        m->V[dst + a] = m->V[src + a];
      }
    }
    return;
  }
  real *a = (real *)malloc(sizeof(real) * (size_t)c->d_model);
  real *k = (real *)malloc(sizeof(real) * (size_t)nkv);
  real *v = (real *)malloc(sizeof(real) * (size_t)nkv);
  project_kv(m, l, x, pos, a, k, v);
  store_kv(m, l, slot, pos, k, v);
  free(a); free(k); free(v);
}

static void embed(const d3o_model *m, int tok, real *x) {
  int d = m->c.d_model;
  for (int e = 0; e < d; ++e) x[e] = bf16_to_real(m->w.embed[(size_t)tok * d + e]);
}

static void head(const d3o_model *m, const real *x, double *logits) {
  const d3o_config *c = &m->c;
  real *a = (real *)malloc(sizeof(real) * (size_t)c->d_model);
  real *y = (real *)malloc(sizeof(real) * (size_t)c->vocab);
  d3o_rmsnorm(x, m->w.final_norm, c->d_model, c->rms_eps, a);
  matvec(m->w.lm_head, c->vocab, c->d_model, a, y);
  for (int r = 0; r < c->vocab; ++r) logits[r] = (double)y[r];
  free(a); free(y);
}

/* Saturation probe (Sec. 3.2, the oracle experiment behind the saturation table):
 * the token a block's output would predict, lm_head(h^i) with the model's final
 * norm, and the confidence softmax gives it.  hidden [d] is a residual-stream
 * state (e.g. a row of d3o_decode_step's trace); logits [vocab] is filled;
 * *token = argmax (lowest index on ties), *confidence = its softmax probability. */
int32_t d3o_probe(const d3o_model *m, const double *hidden, double *logits, int32_t *token,
                  double *confidence) {
  const d3o_config *c = &m->c;
  real *x = (real *)malloc(sizeof(real) * (size_t)c->d_model);
  for (int e = 0; e < c->d_model; ++e) x[e] = (real)hidden[e];
  head(m, x, logits);
  free(x);
  int32_t best = 0;
  for (int32_t r = 1; r < c->vocab; ++r)
    if (logits[r] > logits[best]) best = r;
  double z = 0.0;
  for (int32_t r = 0; r < c->vocab; ++r) z += exp(logits[r] - logits[best]);
  *token = best;
  *confidence = 1.0 / z;
  return 0;
}

/* Initiation phase (Sec. 3.1): every prompt token through all L blocks; the
 * logits of the last position choose T_0.  hidden_out (nullable, [d]) gets the
 * last position's residual stream before the final norm. */
int32_t d3o_prefill(d3o_model *m, int32_t slot, const int32_t *tokens, int32_t n_tokens,
                    double *logits, double *hidden_out) {
  const d3o_config *c = &m->c;
  if (slot < 0 || slot >= c->max_slots || n_tokens < 1 || n_tokens > c->max_seq) return -1;
  for (int t = 0; t < n_tokens; ++t)
    if (tokens[t] < 0 || tokens[t] >= c->vocab) return -1;
  real *x = (real *)malloc(sizeof(real) * (size_t)c->d_model);
  for (int t = 0; t < n_tokens; ++t) {
    embed(m, tokens[t], x);
    for (int l = 0; l < c->n_layers; ++l) block(m, l, x, slot, t);
  }
  m->pos[slot] = n_tokens;
  if (logits) head(m, x, logits);
  if (hidden_out)
    for (int e = 0; e < c->d_model; ++e) hidden_out[e] = (double)x[e];
  free(x);
  return 0;
}

/* Generation phase, one step for a batch of sequences (Sec. 3.4 + Appendix
 * Table "HP description").  Row b feeds token T_{i_b - 1} at its slot's next
 * cache position, runs the blocks outside its window, fills the window's KV
 * per the fill mode, and returns the logits that choose T_{i_b}.
 *   logits  [B][vocab]; hidden (nullable) [B][d] residual stream before the
 *   final norm; trace (nullable) [B][L+1][d] residual stream before block 0
 *   and after every layer. */
static int32_t step_with_depths(d3o_model *m, int32_t B, const int32_t *slots, const int32_t *tokens,
                                const int32_t *depths, double *logits, double *hidden,
                                double *trace);

int32_t d3o_decode_step(d3o_model *m, int32_t B, const int32_t *slots, const int32_t *tokens,
                        const int32_t *gen_index, double alpha, double *logits,
                        double *hidden, double *trace) {
  if (B < 1 || !(alpha > 0.0) || !(alpha <= 1.0)) return -1;
  int32_t *depths = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
  for (int b = 0; b < B; ++b) {
    if (gen_index[b] < 1) { free(depths); return -1; }
    depths[b] = d3o_depth(m->c.n_layers, alpha, gen_index[b]);
  }
  int32_t rc = step_with_depths(m, B, slots, tokens, depths, logits, hidden, trace);
  free(depths);
  return rc;
}

/* The same step with the retained count of every row given by the caller
 * (0 <= depths[b] <= L): whatever schedule produced the counts, the window, the
 * carried hidden state and the KV fill follow the rules above. */
int32_t d3o_decode_step_depths(d3o_model *m, int32_t B, const int32_t *slots, const int32_t *tokens,
                               const int32_t *depths, double *logits, double *hidden,
                               double *trace) {
  if (B < 1) return -1;
  for (int b = 0; b < B; ++b)
    if (depths[b] < 0 || depths[b] > m->c.n_layers) return -1;
  return step_with_depths(m, B, slots, tokens, depths, logits, hidden, trace);
}

static int32_t step_with_depths(d3o_model *m, int32_t B, const int32_t *slots, const int32_t *tokens,
                                const int32_t *depths, double *logits, double *hidden,
                                double *trace) {
  const d3o_config *c = &m->c;
  int L = c->n_layers, d = c->d_model;
  for (int b = 0; b < B; ++b) {
    if (slots[b] < 0 || slots[b] >= c->max_slots) return -1;
    if (tokens[b] < 0 || tokens[b] >= c->vocab) return -1;
    if (m->pos[slots[b]] < 1) return -3;
    if (m->pos[slots[b]] >= c->max_seq) return -2;
    for (int a = 0; a < b; ++a)
      if (slots[a] == slots[b]) return -3;
  }
  real *x = (real *)malloc(sizeof(real) * (size_t)d);
  for (int b = 0; b < B; ++b) {
    int slot = slots[b], pos = m->pos[slot];
    int32_t lo, hi;
    int32_t n = window_of_depth(L, depths[b], c->start_id, c->anchor, &lo, &hi);
    if (n < 0) { free(x); return -1; }
    embed(m, tokens[b], x);
    for (int l = 0; l < L; ++l) {
      if (trace)
        for (int e = 0; e < d; ++e) trace[((size_t)b * (L + 1) + l) * d + e] = (double)x[e];
      if (lo <= l && l < hi)
        fill_kv(m, l, slot, pos, x, lo); /* hidden state passes through unchanged */
      else
        block(m, l, x, slot, pos);
    }
    if (trace)
      for (int e = 0; e < d; ++e) trace[((size_t)b * (L + 1) + L) * d + e] = (double)x[e];
    m->pos[slot] = pos + 1;
    head(m, x, logits + (size_t)b * c->vocab);
    if (hidden)
      for (int e = 0; e < d; ++e) hidden[(size_t)b * d + e] = (double)x[e];
  }
  free(x);
  return 0;
}

/* A decode step written without any schedule code: run exactly the listed
 * blocks, in the order given, on one row; nothing is filled.  Used to check
 * the scheduled step against a hand-truncated stack. */
int32_t d3o_decode_layers(d3o_model *m, int32_t slot, int32_t token, const int32_t *layers,
                          int32_t n_layers_run, double *logits, double *hidden) {
  const d3o_config *c = &m->c;
  if (slot < 0 || slot >= c->max_slots || m->pos[slot] < 1 || m->pos[slot] >= c->max_seq)
    return -1;
  real *x = (real *)malloc(sizeof(real) * (size_t)c->d_model);
  int pos = m->pos[slot];
  embed(m, token, x);
  for (int a = 0; a < n_layers_run; ++a) block(m, layers[a], x, slot, pos);
  m->pos[slot] = pos + 1;
  head(m, x, logits);
  if (hidden)
    for (int e = 0; e < c->d_model; ++e) hidden[e] = (double)x[e];
  free(x);
  return 0;
}

/* Whole-sequence forward at full depth with NO cache: every layer recomputes
 * queries, keys and values of all positions and applies attention with the
 * causal bound t' <= t.  logits_all is [n_tokens][vocab].  Written apart from
 * block(): it must agree with prefill + cached full-depth decode. */
int32_t d3o_forward_nocache(const d3o_model *m, const int32_t *tokens, int32_t n_tokens,
                            double *logits_all) {
  const d3o_config *c = &m->c;
  int d = c->d_model, dh = c->head_dim, Hq = c->n_q_heads, Hkv = c->n_kv_heads, f = c->d_ffn;
  int nq = Hq * dh, nkv = Hkv * dh, T = n_tokens;
  real *X = (real *)malloc(sizeof(real) * (size_t)T * d);
  real *Q = (real *)malloc(sizeof(real) * (size_t)T * nq);
  real *Kc = (real *)malloc(sizeof(real) * (size_t)T * nkv);
  real *Vc = (real *)malloc(sizeof(real) * (size_t)T * nkv);
  real *O = (real *)malloc(sizeof(real) * (size_t)nq);
  real *a = (real *)malloc(sizeof(real) * (size_t)d);
  real *y = (real *)malloc(sizeof(real) * (size_t)d);
  real *g = (real *)malloc(sizeof(real) * (size_t)f);
  real *u = (real *)malloc(sizeof(real) * (size_t)f);
  real *p = (real *)malloc(sizeof(real) * (size_t)T);
  for (int t = 0; t < T; ++t) embed(m, tokens[t], X + (size_t)t * d);
  for (int l = 0; l < c->n_layers; ++l) {
    for (int t = 0; t < T; ++t) {
      d3o_rmsnorm(X + (size_t)t * d, m->w.attn_norm[l], d, c->rms_eps, a);
      matvec(m->w.wq[l], nq, d, a, Q + (size_t)t * nq);
      matvec(m->w.wk[l], nkv, d, a, Kc + (size_t)t * nkv);
      matvec(m->w.wv[l], nkv, d, a, Vc + (size_t)t * nkv);
      for (int h = 0; h < Hq; ++h) d3o_rope(Q + (size_t)t * nq + h * dh, dh, t, c->rope_base);
      for (int h = 0; h < Hkv; ++h) d3o_rope(Kc + (size_t)t * nkv + h * dh, dh, t, c->rope_base);
    }
    for (int t = 0; t < T; ++t) {
      for (int h = 0; h < Hq; ++h) {
        int kvh = h / (Hq / Hkv);
        for (int s = 0; s <= t; ++s) {
          real acc = 0;
          for (int e = 0; e < dh; ++e)
            acc += Q[(size_t)t * nq + h * dh + e] * Kc[(size_t)s * nkv + kvh * dh + e];
          p[s] = acc / (real)sqrt((double)dh);
        }
        d3o_softmax(p, t + 1);
        for (int e = 0; e < dh; ++e) {
          real acc = 0;
          for (int s = 0; s <= t; ++s) acc += p[s] * Vc[(size_t)s * nkv + kvh * dh + e];
          O[h * dh + e] = acc;
        }
      }
      matvec(m->w.wo[l], d, nq, O, y);
      for (int e = 0; e < d; ++e) X[(size_t)t * d + e] += y[e];
    }
    for (int t = 0; t < T; ++t) {
      d3o_rmsnorm(X + (size_t)t * d, m->w.mlp_norm[l], d, c->rms_eps, a);
      matvec(m->w.w_gate[l], f, d, a, g);
      matvec(m->w.w_up[l], f, d, a, u);
      for (int e = 0; e < f; ++e) u[e] = silu(g[e]) * u[e];
      matvec(m->w.w_down[l], d, f, u, y);
      for (int e = 0; e < d; ++e) X[(size_t)t * d + e] += y[e];
    }
  }
  for (int t = 0; t < T; ++t) head(m, X + (size_t)t * d, logits_all + (size_t)t * c->vocab);
  free(X); free(Q); free(Kc); free(Vc); free(O); free(a); free(y); free(g); free(u); free(p);
  return 0;
}

/* lowest index of the maximum */
int32_t d3o_argmax(const double *v, int32_t n) {
  int32_t best = 0;
  for (int32_t a = 1; a < n; ++a)
    if (v[a] > v[best]) best = a;
  return best;
}
