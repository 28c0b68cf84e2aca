/*
 * GLIDE hybrid attention -- CPU oracle (TEST INFRASTRUCTURE, not the product).
 *
 * Plain C, fp64 everywhere, explicit loops, no blocking / fusion / reordering
 * beyond what the definition states.  It shares no code with the CUDA path.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call into this file.
 *
 * What it computes (paper Sec. III-B "GLIDE Attention", Eq. 7 and the two
 * component equations that follow it; Sec. II "Linearized Attention";
 * appendix Eq. 1-6):
 *
 *   position t (0-indexed) of one sequence in one layer with window w:
 *     W_t = { j : max(0, t-w+1) <= j <= t }     newest w tokens, current included
 *     E_t = { j : 0 <= j <= t-w }               everything older ("evicted")
 *     a_j = exp(scale * <q_t, k_j>)             j in W_t   (appendix Eq. 1)
 *     c_j = <phi(q_t), phi(k_j)>                j in E_t   (Eq. 5), phi = softmax over
 *                                               the d entries of the vector
 *     O_t = (sum_W a_j v_j + sum_E c_j v_j) / (sum_W a_j + sum_E c_j)
 *   i.e. the "(+)" operator read as one shared normaliser (the outputs of the two
 *   parts weighted by their own denominators).
 *
 * Two forms:
 *   form B  glide_oracle_bruteforce(): the sums above over the full history.
 *   form A  glide_oracle_cell: the stateful restatement -- a ring buffer of the
 *           last w keys/values plus the recurrent state S = sum_E phi(k_j) v_j^T,
 *           z = sum_E phi(k_j) (Sec. II recurrences), with decode() (one token,
 *           incremental fold) and prefill() (many tokens, explicit sums).
 *
 * Alternative merges (appendix "(b) Retention-based SWA", the two hybrid equations): merge = 1 adds the
 * separately normalised linear term over the evicted tokens and the separately normalised window softmax,
 *   O_t = phi(q) S_{t-w} / phi(q) z_{t-w} + sum_W a_j v_j / sum_W a_j ;
 * merge = 2 is the same sum with the state holding every token up to t (S_t, z_t).  A term whose token set is
 * empty is taken as zero (the paper is silent; its quotient would be 0/0).  merge = 0 is the shared normaliser.
 *
 * Feature maps (the appendix' "Linear Attention" lists the kernels the method accepts; Sec. III-B: the default is
 * the parameter-free softmax): phi kind 0 is phi(x) = softmax over the d entries of x, feature dimension d.  Kind 1
 * is the learned map of the Hedgehog / LoLCATs line the paper builds on, whose formula the paper does not print
 * (a reading): with a d x d matrix W per head, y = W^T x (y_j = sum_i x_i W[i][j]),
 *   phi_W(x) = [ softmax(y) ; softmax(-y) ],   feature dimension 2d,
 * one matrix per query head for the queries and one per KV head for the keys.  S is then [2d][d], z [2d].
 *
 * Gated recurrence (Sec. III-B "GLA-style gating mechanisms"; the paper gives no formula: a reading): every token
 * brings a decay gamma in (0, 1] per KV head, and the state decays by the gate of the token that enters it,
 *   S <- gamma_j S + phi(k_j) v_j^T,   z <- gamma_j z + phi(k_j),
 * so a token i of the state weighs prod over the later-entered tokens j of gamma_j.  gamma == 1 is the method as
 * printed.  The gates of the window's tokens wait in the ring with their keys and values.
 *
 * Parity pins (tests, CPU only): form A vs form B; w >= n vs a library causal
 * softmax attention; w = 0 vs matrix-form linear attention; the closed form for
 * q = k = 0; convexity; decode == prefill.  Random-input output VALUES have no
 * printed worked example in the paper: beyond those pins they are
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* phi(x) = softmax over the d entries of x (Sec. III-B: default kernel). */
static void phi_softmax(const double *x, int d, double *out) {
  double mx = x[0];
  for (int r = 1; r < d; ++r)
    if (x[r] > mx) mx = x[r];
  double sum = 0.0;
  for (int r = 0; r < d; ++r) {
    out[r] = exp(x[r] - mx);
    sum += out[r];
  }
  for (int r = 0; r < d; ++r) out[r] /= sum;
}

/* Feature dimension of a map kind. */
static int phi_dim(int kind, int d) { return kind == 1 ? 2 * d : d; }

/* phi of one vector x [d] -> out [phi_dim].  kind 1: W [d][d] of the vector's head, y = W^T x, the two halves
 * softmax(y) and softmax(-y). */
static void phi_apply(int kind, const double *W, const double *x, int d, double *out) {
  if (kind == 0) {
    phi_softmax(x, d, out);
    return;
  }
  double *y = (double *)malloc(sizeof(double) * d);
  for (int j = 0; j < d; ++j) {
    double acc = 0.0;
    for (int i = 0; i < d; ++i) acc += x[i] * W[(size_t)i * d + j];
    y[j] = acc;
  }
  phi_softmax(y, d, out);
  for (int j = 0; j < d; ++j) y[j] = -y[j];
  phi_softmax(y, d, out + d);
  free(y);
}

static double dot(const double *a, const double *b, int d) {
  double s = 0.0;
  for (int r = 0; r < d; ++r) s += a[r] * b[r];
  return s;
}

/* The merge of the two parts.  numw/denw: window sums already multiplied by exp(-M); numl/denl: linear sums.
 * merge 0: one shared normaliser (Sec. III-B); merge 1, 2: the sum of the two separately normalised terms
 * (appendix hybrid equations), an empty term counting as zero. */
static void combine(int merge, int d, double M, const double *numw, double denw, const double *numl,
                    double denl, double *o) {
  if (merge == 0) {
    double eM = exp(-M);
    for (int c = 0; c < d; ++c) o[c] = (numw[c] + eM * numl[c]) / (denw + eM * denl);
    return;
  }
  for (int c = 0; c < d; ++c) {
    double x = 0.0;
    if (denw > 0.0) x += numw[c] / denw;
    if (denl > 0.0) x += numl[c] / denl;
    o[c] = x;
  }
}

/* ------------------------------------------------------------------------- */
/* Form B: brute force over the full history.                                 */
/* q [T][H][d], k,v [T][Hkv][d], out [n_sel][H][d]; sel = positions to        */
/* evaluate (NULL: all T positions, n_sel ignored).                           */
/* ------------------------------------------------------------------------- */
/* phi_kind, wq [H][d][d], wk [Hkv][d][d]: the feature map (kind 0: both NULL).  gate [T][Hkv] or NULL: the decay  */
/* each token brings; the linear weight of token j at position t is c_j times the gates of the tokens that entered  */
/* the state after j, i.e. of tokens j+1 .. t-delay.                                                                  */
void glide_oracle_bruteforce_ex(int64_t T, int H, int Hkv, int d, int64_t w, double scale, int merge,
                                const int32_t *q_to_kv, const double *q, const double *k,
                                const double *v, int64_t n_sel, const int64_t *sel, double *out,
                                int phi_kind, const double *wq, const double *wk, const double *gate) {
  int64_t count = sel ? n_sel : T;
  int64_t delay = merge == 2 ? 0 : w; /* the linear term covers tokens j <= t - delay */
  int dp = phi_dim(phi_kind, d);
  double *phiq = (double *)malloc(sizeof(double) * dp);
  double *phik = (double *)malloc(sizeof(double) * dp);
  double *num = (double *)malloc(sizeof(double) * d);
  double *numl = (double *)malloc(sizeof(double) * d);
  for (int64_t si = 0; si < count; ++si) {
    int64_t t = sel ? sel[si] : si;
    for (int h = 0; h < H; ++h) {
      int g = q_to_kv[h];
      const double *qt = q + ((size_t)t * H + h) * d;
      int64_t w_lo = t - w + 1;
      if (w_lo < 0) w_lo = 0;
      /* M = max(0, max_W scale<q,k_j>): multiplying numerator and denominator by
       * exp(-M) is an identity that keeps exp() in range. */
      double M = 0.0;
      for (int64_t j = w_lo; j <= t; ++j) {
        double s = scale * dot(qt, k + ((size_t)j * Hkv + g) * d, d);
        if (s > M) M = s;
      }
      double den = 0.0;
      for (int c = 0; c < d; ++c) num[c] = 0.0;
      for (int64_t j = w_lo; j <= t; ++j) { /* empty when w == 0 */
        const double *kj = k + ((size_t)j * Hkv + g) * d;
        const double *vj = v + ((size_t)j * Hkv + g) * d;
        double a = exp(scale * dot(qt, kj, d) - M);
        den += a;
        for (int c = 0; c < d; ++c) num[c] += a * vj[c];
      }
      phi_apply(phi_kind, wq ? wq + (size_t)h * d * d : NULL, qt, d, phiq);
      double denl = 0.0;
      for (int c = 0; c < d; ++c) numl[c] = 0.0;
      for (int64_t j = 0; j <= t - delay; ++j) { /* empty when t < delay */
        const double *kj = k + ((size_t)j * Hkv + g) * d;
        const double *vj = v + ((size_t)j * Hkv + g) * d;
        phi_apply(phi_kind, wk ? wk + (size_t)g * d * d : NULL, kj, d, phik);
        double c_j = dot(phiq, phik, dp);
        if (gate)
          for (int64_t m = j + 1; m <= t - delay; ++m) c_j *= gate[(size_t)m * Hkv + g];
        denl += c_j;
        for (int c = 0; c < d; ++c) numl[c] += c_j * vj[c];
      }
      combine(merge, d, M, num, den, numl, denl, out + ((size_t)si * H + h) * d);
    }
  }
  free(phiq);
  free(phik);
  free(num);
  free(numl);
}

void glide_oracle_bruteforce(int64_t T, int H, int Hkv, int d, int64_t w, double scale, int merge,
                             const int32_t *q_to_kv, const double *q, const double *k,
                             const double *v, int64_t n_sel, const int64_t *sel, double *out) {
  glide_oracle_bruteforce_ex(T, H, Hkv, d, w, scale, merge, q_to_kv, q, k, v, n_sel, sel, out, 0, NULL, NULL, NULL);
}

/* ------------------------------------------------------------------------- */
/* Form A: one (layer, sequence) cell with ring + recurrent state.            */
/* ------------------------------------------------------------------------- */
typedef struct glide_oracle_cell {
  int H, Hkv, d;
  int64_t w;     /* window; ring capacity is exactly w (0: no ring) */
  int merge;     /* 0 shared normaliser, 1 / 2 the appendix' sums of two normalised terms */
  int64_t delay; /* a token enters the state `delay` steps after it arrives: w, or 0 for merge 2 */
  double scale;
  int32_t *q_to_kv;
  int phi_kind;  /* 0 softmax over the features; 1 learned projection, two softmax halves */
  int dp;        /* feature dimension: d or 2d */
  double *wq;    /* kind 1: [H][d][d] */
  double *wk;    /* kind 1: [Hkv][d][d] */
  int64_t n;     /* tokens absorbed so far */
  double *Kr;    /* [Hkv][w][d] */
  double *Vr;    /* [Hkv][w][d] */
  double *Gr;    /* [Hkv][w]  gates of the ring's tokens (1 when the caller gives none) */
  double *S;     /* [Hkv][dp][d]   S[r][c] = sum (decay) phi(k)_r v_c */
  double *z;     /* [Hkv][dp] */
} glide_oracle_cell;

glide_oracle_cell *glide_oracle_cell_new(int H, int Hkv, int d, int64_t w, double scale, int merge,
                                         const int32_t *q_to_kv) {
  glide_oracle_cell *c = (glide_oracle_cell *)calloc(1, sizeof(*c));
  c->H = H;
  c->Hkv = Hkv;
  c->d = d;
  c->w = w;
  c->merge = merge;
  c->delay = merge == 2 ? 0 : w;
  c->scale = scale;
  c->q_to_kv = (int32_t *)malloc(sizeof(int32_t) * H);
  memcpy(c->q_to_kv, q_to_kv, sizeof(int32_t) * H);
  c->phi_kind = 0;
  c->dp = d;
  size_t slots = (size_t)Hkv * (size_t)(w > 0 ? w : 1);
  c->Kr = (double *)calloc(slots * d, sizeof(double));
  c->Vr = (double *)calloc(slots * d, sizeof(double));
  c->Gr = (double *)calloc(slots, sizeof(double));
  c->S = (double *)calloc((size_t)Hkv * d * d, sizeof(double));
  c->z = (double *)calloc((size_t)Hkv * d, sizeof(double));
  return c;
}

/* Selects the feature map of an EMPTY cell: kind 1 takes wq [H][d][d] and wk [Hkv][d][d] (copied). */
void glide_oracle_cell_set_phi(glide_oracle_cell *c, int kind, const double *wq, const double *wk) {
  int d = c->d;
  c->phi_kind = kind;
  c->dp = phi_dim(kind, d);
  free(c->wq);
  free(c->wk);
  c->wq = c->wk = NULL;
  if (kind == 1) {
    c->wq = (double *)malloc(sizeof(double) * (size_t)c->H * d * d);
    c->wk = (double *)malloc(sizeof(double) * (size_t)c->Hkv * d * d);
    memcpy(c->wq, wq, sizeof(double) * (size_t)c->H * d * d);
    memcpy(c->wk, wk, sizeof(double) * (size_t)c->Hkv * d * d);
  }
  free(c->S);
  free(c->z);
  c->S = (double *)calloc((size_t)c->Hkv * c->dp * d, sizeof(double));
  c->z = (double *)calloc((size_t)c->Hkv * c->dp, sizeof(double));
}

int glide_oracle_cell_phi_dim(const glide_oracle_cell *c) { return c->dp; }

void glide_oracle_cell_free(glide_oracle_cell *c) {
  if (!c) return;
  free(c->q_to_kv);
  free(c->wq);
  free(c->wk);
  free(c->Kr);
  free(c->Vr);
  free(c->Gr);
  free(c->S);
  free(c->z);
  free(c);
}

void glide_oracle_cell_reset(glide_oracle_cell *c) {
  size_t slots = (size_t)c->Hkv * (size_t)(c->w > 0 ? c->w : 1);
  memset(c->Kr, 0, slots * c->d * sizeof(double));
  memset(c->Vr, 0, slots * c->d * sizeof(double));
  memset(c->Gr, 0, slots * sizeof(double));
  memset(c->S, 0, (size_t)c->Hkv * c->dp * c->d * sizeof(double));
  memset(c->z, 0, (size_t)c->Hkv * c->dp * sizeof(double));
  c->n = 0;
}

static const double *cell_wq(const glide_oracle_cell *c, int h) {
  return c->wq ? c->wq + (size_t)h * c->d * c->d : NULL;
}
static const double *cell_wk(const glide_oracle_cell *c, int g) {
  return c->wk ? c->wk + (size_t)g * c->d * c->d : NULL;
}

/* S_g <- gamma S_g + phi(k) v^T ; z_g <- gamma z_g + phi(k)   (Sec. II recurrences; gamma = 1 without gating) */
static void fold(glide_oracle_cell *c, int g, const double *kv_k, const double *kv_v, double gamma,
                 double *phik /* scratch [dp] */) {
  int d = c->d, dp = c->dp;
  phi_apply(c->phi_kind, cell_wk(c, g), kv_k, d, phik);
  double *S = c->S + (size_t)g * dp * d;
  double *z = c->z + (size_t)g * dp;
  for (int r = 0; r < dp; ++r) {
    z[r] = gamma * z[r] + phik[r];
    for (int col = 0; col < d; ++col) S[(size_t)r * d + col] = gamma * S[(size_t)r * d + col] + phik[r] * kv_v[col];
  }
}

/* Bookkeeping step shared by nothing else: advance KV head g by one token (gamma: the token's gate). */
static void append_token(glide_oracle_cell *c, int g, int64_t t, const double *k,
                         const double *v, double gamma, double *phik) {
  int d = c->d;
  int64_t w = c->w;
  if (c->delay == 0) fold(c, g, k, v, gamma, phik); /* no ring (w = 0) or the all-token state: token t enters the state now */
  if (w == 0) return;
  int64_t slot = t % w;
  double *Kslot = c->Kr + ((size_t)g * w + slot) * d;
  double *Vslot = c->Vr + ((size_t)g * w + slot) * d;
  double *Gslot = c->Gr + (size_t)g * w + slot;
  if (c->delay > 0 && t >= w) fold(c, g, Kslot, Vslot, *Gslot, phik); /* that slot holds token t-w, which leaves the window */
  memcpy(Kslot, k, sizeof(double) * d);
  memcpy(Vslot, v, sizeof(double) * d);
  *Gslot = gamma;
}

/* Readout for query head h at position t, AFTER token t was appended. */
static void readout(const glide_oracle_cell *c, int h, int64_t t, const double *qt,
                    double *o, double *phiq /* [dp] */, double *num) {
  int d = c->d, dp = c->dp;
  int64_t w = c->w;
  int g = c->q_to_kv[h];
  int64_t w_lo = t - w + 1;
  if (w_lo < 0) w_lo = 0;
  const double *Kr = c->Kr + (size_t)g * (w > 0 ? w : 1) * d;
  const double *Vr = c->Vr + (size_t)g * (w > 0 ? w : 1) * d;
  double M = 0.0;
  for (int64_t j = w_lo; j <= t && w > 0; ++j) {
    double s = c->scale * dot(qt, Kr + (size_t)(j % w) * d, d);
    if (s > M) M = s;
  }
  double den = 0.0;
  for (int col = 0; col < d; ++col) num[col] = 0.0;
  for (int64_t j = w_lo; j <= t && w > 0; ++j) {
    const double *kj = Kr + (size_t)(j % w) * d;
    const double *vj = Vr + (size_t)(j % w) * d;
    double a = exp(c->scale * dot(qt, kj, d) - M);
    den += a;
    for (int col = 0; col < d; ++col) num[col] += a * vj[col];
  }
  /* linear part: phi(q) S and phi(q) z on the state that already holds its token set */
  phi_apply(c->phi_kind, cell_wq(c, h), qt, d, phiq);
  const double *S = c->S + (size_t)g * dp * d;
  const double *z = c->z + (size_t)g * dp;
  double *numl = (double *)malloc(sizeof(double) * d);
  double denl = 0.0;
  for (int col = 0; col < d; ++col) numl[col] = 0.0;
  for (int r = 0; r < dp; ++r) {
    denl += phiq[r] * z[r];
    for (int col = 0; col < d; ++col) numl[col] += phiq[r] * S[(size_t)r * d + col];
  }
  combine(c->merge, d, M, num, den, numl, denl, o);
  free(numl);
}

/* One decode step for the heads of KV head g only (used for threading).  gate: [Hkv] or NULL. */
static void decode_group(glide_oracle_cell *c, int g, const double *q, const double *k,
                         const double *v, const double *gate, double *out) {
  int d = c->d, dp = c->dp;
  int64_t t = c->n;
  double *tmp = (double *)malloc(sizeof(double) * (2 * dp + d));
  append_token(c, g, t, k + (size_t)g * d, v + (size_t)g * d, gate ? gate[g] : 1.0, tmp);
  for (int h = 0; h < c->H; ++h) {
    if (c->q_to_kv[h] != g) continue;
    readout(c, h, t, q + (size_t)h * d, out + (size_t)h * d, tmp + dp, tmp + 2 * dp);
  }
  free(tmp);
}

/* decode: q [H][d], k,v [Hkv][d], gate [Hkv] or NULL -> out [H][d]; n += 1 */
void glide_oracle_cell_decode_ex(glide_oracle_cell *c, const double *q, const double *k,
                                 const double *v, const double *gate, double *out) {
  for (int g = 0; g < c->Hkv; ++g) decode_group(c, g, q, k, v, gate, out);
  c->n += 1;
}

void glide_oracle_cell_decode(glide_oracle_cell *c, const double *q, const double *k,
                              const double *v, double *out) {
  glide_oracle_cell_decode_ex(c, q, k, v, NULL, out);
}

/* One decode step of many cells (layers x sequences), threaded over
 * (cell, KV head) units.  q [n_cells][H][d], k,v [n_cells][Hkv][d], gate [n_cells][Hkv] or NULL. */
int glide_oracle_stack_decode_ex(glide_oracle_cell **cells, int64_t n_cells, const double *q,
                                 const double *k, const double *v, const double *gate, double *out, int n_threads) {
  if (n_cells <= 0) return 0;
  int H = cells[0]->H, Hkv = cells[0]->Hkv, d = cells[0]->d;
  int used = 1;
  int64_t units = n_cells * Hkv;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel
  {
#pragma omp single
    used = omp_get_num_threads();
#pragma omp for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
      int64_t ci = u / Hkv;
      int g = (int)(u % Hkv);
      decode_group(cells[ci], g, q + (size_t)ci * H * d, k + (size_t)ci * Hkv * d,
                   v + (size_t)ci * Hkv * d, gate ? gate + (size_t)ci * Hkv : NULL, out + (size_t)ci * H * d);
    }
  }
#else
  (void)n_threads;
  for (int64_t u = 0; u < units; ++u) {
    int64_t ci = u / Hkv;
    int g = (int)(u % Hkv);
    decode_group(cells[ci], g, q + (size_t)ci * H * d, k + (size_t)ci * Hkv * d,
                 v + (size_t)ci * Hkv * d, gate ? gate + (size_t)ci * Hkv : NULL, out + (size_t)ci * H * d);
  }
#endif
  for (int64_t ci = 0; ci < n_cells; ++ci) cells[ci]->n += 1;
  return used;
}

int glide_oracle_stack_decode(glide_oracle_cell **cells, int64_t n_cells, const double *q,
                              const double *k, const double *v, double *out, int n_threads) {
  return glide_oracle_stack_decode_ex(cells, n_cells, q, k, v, NULL, out, n_threads);
}

/*
 * prefill: append T tokens.  q [T][H][d] (may be NULL when n_sel == 0),
 * k,v [T][Hkv][d], gate [T][Hkv] or NULL, out [n_sel][H][d] for the call-relative positions in sel
 * (sel == NULL and n_sel < 0: all T positions).
 *
 * Outputs are NOT produced by repeated decode steps: each selected position is
 * evaluated from explicit sums -- the window over ring-or-call tokens, the
 * evicted set as (state at call start, decayed by the gates of the tokens that entered since) +
 * (explicit sum over the tokens that left the window since the call started, each with the gates of
 * the tokens that entered after it).  The state is then rebuilt by its
 * definition: the tokens that left the window during the call are folded in order,
 * ring slot s = the newest token j with j mod w == s.
 */
void glide_oracle_cell_prefill_ex(glide_oracle_cell *c, int64_t T, const double *q,
                                  const double *k, const double *v, const double *gate, int64_t n_sel,
                                  const int64_t *sel, double *out) {
  int d = c->d, dp = c->dp, H = c->H, Hkv = c->Hkv;
  int64_t w = c->w, n0 = c->n, delay = c->delay;
  int64_t count = (sel == NULL && n_sel < 0) ? T : n_sel;
  double *phiq = (double *)malloc(sizeof(double) * dp);
  double *phik = (double *)malloc(sizeof(double) * dp);
  double *num = (double *)malloc(sizeof(double) * d);
  double *numl = (double *)malloc(sizeof(double) * d);

/* token j (absolute index) of KV head g: from the call if j >= n0, else from the ring */
#define TOK_K(j, g) ((j) >= n0 ? k + ((size_t)((j)-n0) * Hkv + (g)) * d \
                               : c->Kr + ((size_t)(g) * w + (size_t)((j) % w)) * d)
#define TOK_V(j, g) ((j) >= n0 ? v + ((size_t)((j)-n0) * Hkv + (g)) * d \
                               : c->Vr + ((size_t)(g) * w + (size_t)((j) % w)) * d)
#define TOK_G(j, g) ((j) >= n0 ? (gate ? gate[(size_t)((j)-n0) * Hkv + (g)] : 1.0) \
                               : c->Gr[(size_t)(g) * w + (size_t)((j) % w)])

  for (int64_t si = 0; si < count; ++si) {
    int64_t rel = sel ? sel[si] : si;
    int64_t t = n0 + rel;
    for (int h = 0; h < H; ++h) {
      int g = c->q_to_kv[h];
      const double *qt = q + ((size_t)rel * H + h) * d;
      int64_t w_lo = t - w + 1;
      if (w_lo < 0) w_lo = 0;
      double M = 0.0;
      for (int64_t j = w_lo; j <= t; ++j) {
        double s = c->scale * dot(qt, TOK_K(j, g), d);
        if (s > M) M = s;
      }
      double den = 0.0;
      for (int col = 0; col < d; ++col) num[col] = 0.0;
      for (int64_t j = w_lo; j <= t; ++j) {
        double a = exp(c->scale * dot(qt, TOK_K(j, g), d) - M);
        const double *vj = TOK_V(j, g);
        den += a;
        for (int col = 0; col < d; ++col) num[col] += a * vj[col];
      }
      phi_apply(c->phi_kind, cell_wq(c, h), qt, d, phiq);
      /* entered the state since the call started: tokens e_lo .. t-delay */
      int64_t e_lo = n0 - delay;
      if (e_lo < 0) e_lo = 0;
      /* in the state before the call started, decayed by the gates of everything that entered since */
      double decay0 = 1.0;
      for (int64_t m = e_lo; m <= t - delay; ++m) decay0 *= TOK_G(m, g);
      const double *S = c->S + (size_t)g * dp * d;
      const double *z = c->z + (size_t)g * dp;
      double denl = 0.0;
      for (int col = 0; col < d; ++col) numl[col] = 0.0;
      for (int r = 0; r < dp; ++r) {
        denl += decay0 * phiq[r] * z[r];
        for (int col = 0; col < d; ++col) numl[col] += decay0 * phiq[r] * S[(size_t)r * d + col];
      }
      for (int64_t j = e_lo; j <= t - delay; ++j) {
        phi_apply(c->phi_kind, cell_wk(c, g), TOK_K(j, g), d, phik);
        double c_j = dot(phiq, phik, dp);
        for (int64_t m = j + 1; m <= t - delay; ++m) c_j *= TOK_G(m, g);
        const double *vj = TOK_V(j, g);
        denl += c_j;
        for (int col = 0; col < d; ++col) numl[col] += c_j * vj[col];
      }
      combine(c->merge, d, M, num, den, numl, denl, out + ((size_t)si * H + h) * d);
    }
  }

  /* state by definition: fold tokens [max(0,n0-delay), n0+T-delay) in order ... */
  int64_t n1 = n0 + T;
  for (int g = 0; g < Hkv; ++g) {
    int64_t e_lo = n0 - delay;
    if (e_lo < 0) e_lo = 0;
    for (int64_t j = e_lo; j < n1 - delay; ++j) fold(c, g, TOK_K(j, g), TOK_V(j, g), TOK_G(j, g), phik);
  }
  /* ... then the ring: slot s holds the newest token j < n1 with j mod w == s.
   * Only call tokens need writing; older survivors are already in place. */
  if (w > 0) {
    int64_t first = n1 - w;
    if (first < n0) first = n0;
    for (int g = 0; g < Hkv; ++g)
      for (int64_t j = first; j < n1; ++j) {
        memcpy(c->Kr + ((size_t)g * w + (size_t)(j % w)) * d, k + ((size_t)(j - n0) * Hkv + g) * d,
               sizeof(double) * d);
        memcpy(c->Vr + ((size_t)g * w + (size_t)(j % w)) * d, v + ((size_t)(j - n0) * Hkv + g) * d,
               sizeof(double) * d);
        c->Gr[(size_t)g * w + (size_t)(j % w)] = gate ? gate[(size_t)(j - n0) * Hkv + g] : 1.0;
      }
  }
#undef TOK_K
#undef TOK_V
#undef TOK_G
  c->n = n1;
  free(phiq);
  free(phik);
  free(num);
  free(numl);
}

void glide_oracle_cell_prefill(glide_oracle_cell *c, int64_t T, const double *q,
                               const double *k, const double *v, int64_t n_sel,
                               const int64_t *sel, double *out) {
  glide_oracle_cell_prefill_ex(c, T, q, k, v, NULL, n_sel, sel, out);
}

/* Bookkeeping that the GPU path must reproduce bit-exactly. */
void glide_oracle_cell_info(const glide_oracle_cell *c, int64_t *n, int64_t *count,
                            int64_t *head_slot, int64_t *n_evicted) {
  *n = c->n;
  *count = c->n < c->w ? c->n : c->w;
  *head_slot = c->w > 0 ? c->n % c->w : 0;
  *n_evicted = c->n > c->w ? c->n - c->w : 0;
}

/* token index held by each ring slot (-1: empty); tok [w] */
void glide_oracle_cell_slot_tokens(const glide_oracle_cell *c, int64_t *tok) {
  for (int64_t s = 0; s < c->w; ++s) tok[s] = -1;
  int64_t lo = c->n - c->w;
  if (lo < 0) lo = 0;
  for (int64_t j = lo; j < c->n; ++j) tok[j % c->w] = j; /* the last w tokens, each in slot j mod w */
}

/* Copies of the state: ringK, ringV [Hkv][w][d]; S [Hkv][dp][d]; z [Hkv][dp] (dp = feature dimension). Any may be NULL. */
void glide_oracle_cell_export(const glide_oracle_cell *c, double *ringK, double *ringV,
                              double *S, double *z) {
  size_t ring = (size_t)c->Hkv * (size_t)c->w * c->d;
  if (ringK && ring) memcpy(ringK, c->Kr, ring * sizeof(double));
  if (ringV && ring) memcpy(ringV, c->Vr, ring * sizeof(double));
  if (S) memcpy(S, c->S, (size_t)c->Hkv * c->dp * c->d * sizeof(double));
  if (z) memcpy(z, c->z, (size_t)c->Hkv * c->dp * sizeof(double));
}

/* The gates of the ring's tokens: gates [Hkv][w]. */
void glide_oracle_cell_export_gates(const glide_oracle_cell *c, double *gates) {
  size_t slots = (size_t)c->Hkv * (size_t)c->w;
  if (gates && slots) memcpy(gates, c->Gr, slots * sizeof(double));
}

int glide_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
