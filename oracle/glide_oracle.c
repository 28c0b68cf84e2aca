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
void glide_oracle_bruteforce(int64_t T, int H, int Hkv, int d, int64_t w, double scale, int merge,
                             const int32_t *q_to_kv, const double *q, const double *k,
                             const double *v, int64_t n_sel, const int64_t *sel, double *out) {
  int64_t count = sel ? n_sel : T;
  int64_t delay = merge == 2 ? 0 : w; /* the linear term covers tokens j <= t - delay */
  double *phiq = (double *)malloc(sizeof(double) * d);
  double *phik = (double *)malloc(sizeof(double) * d);
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
      phi_softmax(qt, d, phiq);
      double denl = 0.0;
      for (int c = 0; c < d; ++c) numl[c] = 0.0;
      for (int64_t j = 0; j <= t - delay; ++j) { /* empty when t < delay */
        const double *kj = k + ((size_t)j * Hkv + g) * d;
        const double *vj = v + ((size_t)j * Hkv + g) * d;
        phi_softmax(kj, d, phik);
        double c_j = dot(phiq, phik, d);
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
  int64_t n;     /* tokens absorbed so far */
  double *Kr;    /* [Hkv][w][d] */
  double *Vr;    /* [Hkv][w][d] */
  double *S;     /* [Hkv][d][d]   S[r][c] = sum phi(k)_r v_c */
  double *z;     /* [Hkv][d] */
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
  size_t ring = (size_t)Hkv * (size_t)(w > 0 ? w : 1) * d;
  c->Kr = (double *)calloc(ring, sizeof(double));
  c->Vr = (double *)calloc(ring, sizeof(double));
  c->S = (double *)calloc((size_t)Hkv * d * d, sizeof(double));
  c->z = (double *)calloc((size_t)Hkv * d, sizeof(double));
  return c;
}

void glide_oracle_cell_free(glide_oracle_cell *c) {
  if (!c) return;
  free(c->q_to_kv);
  free(c->Kr);
  free(c->Vr);
  free(c->S);
  free(c->z);
  free(c);
}

void glide_oracle_cell_reset(glide_oracle_cell *c) {
  size_t ring = (size_t)c->Hkv * (size_t)(c->w > 0 ? c->w : 1) * c->d;
  memset(c->Kr, 0, ring * sizeof(double));
  memset(c->Vr, 0, ring * sizeof(double));
  memset(c->S, 0, (size_t)c->Hkv * c->d * c->d * sizeof(double));
  memset(c->z, 0, (size_t)c->Hkv * c->d * sizeof(double));
  c->n = 0;
}

/* S_g += phi(k) v^T ; z_g += phi(k)   (Sec. II recurrences) */
static void fold(glide_oracle_cell *c, int g, const double *kv_k, const double *kv_v,
                 double *phik /* scratch [d] */) {
  int d = c->d;
  phi_softmax(kv_k, d, phik);
  double *S = c->S + (size_t)g * d * d;
  double *z = c->z + (size_t)g * d;
  for (int r = 0; r < d; ++r) {
    z[r] += phik[r];
    for (int col = 0; col < d; ++col) S[(size_t)r * d + col] += phik[r] * kv_v[col];
  }
}

/* Bookkeeping step shared by nothing else: advance KV head g by one token. */
static void append_token(glide_oracle_cell *c, int g, int64_t t, const double *k,
                         const double *v, double *phik) {
  int d = c->d;
  int64_t w = c->w;
  if (c->delay == 0) fold(c, g, k, v, phik); /* no ring (w = 0) or the all-token state: token t enters the state now */
  if (w == 0) return;
  int64_t slot = t % w;
  double *Kslot = c->Kr + ((size_t)g * w + slot) * d;
  double *Vslot = c->Vr + ((size_t)g * w + slot) * d;
  if (c->delay > 0 && t >= w) fold(c, g, Kslot, Vslot, phik); /* that slot holds token t-w, which leaves the window */
  memcpy(Kslot, k, sizeof(double) * d);
  memcpy(Vslot, v, sizeof(double) * d);
}

/* Readout for query head h at position t, AFTER token t was appended. */
static void readout(const glide_oracle_cell *c, int h, int64_t t, const double *qt,
                    double *o, double *phiq, double *num) {
  int d = c->d;
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
  phi_softmax(qt, d, phiq);
  const double *S = c->S + (size_t)g * d * d;
  const double *z = c->z + (size_t)g * d;
  double *numl = (double *)malloc(sizeof(double) * d);
  double denl = 0.0;
  for (int col = 0; col < d; ++col) numl[col] = 0.0;
  for (int r = 0; r < d; ++r) {
    denl += phiq[r] * z[r];
    for (int col = 0; col < d; ++col) numl[col] += phiq[r] * S[(size_t)r * d + col];
  }
  combine(c->merge, d, M, num, den, numl, denl, o);
  free(numl);
}

/* One decode step for the heads of KV head g only (used for threading). */
static void decode_group(glide_oracle_cell *c, int g, const double *q, const double *k,
                         const double *v, double *out) {
  int d = c->d;
  int64_t t = c->n;
  double *tmp = (double *)malloc(sizeof(double) * 3 * d);
  append_token(c, g, t, k + (size_t)g * d, v + (size_t)g * d, tmp);
  for (int h = 0; h < c->H; ++h) {
    if (c->q_to_kv[h] != g) continue;
    readout(c, h, t, q + (size_t)h * d, out + (size_t)h * d, tmp + d, tmp + 2 * d);
  }
  free(tmp);
}

/* decode: q [H][d], k,v [Hkv][d] -> out [H][d]; n += 1 */
void glide_oracle_cell_decode(glide_oracle_cell *c, const double *q, const double *k,
                              const double *v, double *out) {
  for (int g = 0; g < c->Hkv; ++g) decode_group(c, g, q, k, v, out);
  c->n += 1;
}

/* One decode step of many cells (layers x sequences), threaded over
 * (cell, KV head) units.  q [n_cells][H][d], k,v [n_cells][Hkv][d]. */
int glide_oracle_stack_decode(glide_oracle_cell **cells, int64_t n_cells, const double *q,
                              const double *k, const double *v, double *out, int n_threads) {
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
                   v + (size_t)ci * Hkv * d, out + (size_t)ci * H * d);
    }
  }
#else
  (void)n_threads;
  for (int64_t u = 0; u < units; ++u) {
    int64_t ci = u / Hkv;
    int g = (int)(u % Hkv);
    decode_group(cells[ci], g, q + (size_t)ci * H * d, k + (size_t)ci * Hkv * d,
                 v + (size_t)ci * Hkv * d, out + (size_t)ci * H * d);
  }
#endif
  for (int64_t ci = 0; ci < n_cells; ++ci) cells[ci]->n += 1;
  return used;
}

/*
 * prefill: append T tokens.  q [T][H][d] (may be NULL when n_sel == 0),
 * k,v [T][Hkv][d], out [n_sel][H][d] for the call-relative positions in sel
 * (sel == NULL and n_sel < 0: all T positions).
 *
 * Outputs are NOT produced by repeated decode steps: each selected position is
 * evaluated from explicit sums -- the window over ring-or-call tokens, the
 * evicted set as (state at call start) + (explicit sum over the tokens that
 * left the window since the call started).  The state is then rebuilt by its
 * definition: S,z += sum over the tokens that left the window during the call,
 * ring slot s = the newest token j with j mod w == s.
 */
void glide_oracle_cell_prefill(glide_oracle_cell *c, int64_t T, const double *q,
                               const double *k, const double *v, int64_t n_sel,
                               const int64_t *sel, double *out) {
  int d = c->d, H = c->H, Hkv = c->Hkv;
  int64_t w = c->w, n0 = c->n, delay = c->delay;
  int64_t count = (sel == NULL && n_sel < 0) ? T : n_sel;
  double *phiq = (double *)malloc(sizeof(double) * d);
  double *phik = (double *)malloc(sizeof(double) * d);
  double *num = (double *)malloc(sizeof(double) * d);
  double *numl = (double *)malloc(sizeof(double) * d);

/* token j (absolute index) of KV head g: from the call if j >= n0, else from the ring */
#define TOK_K(j, g) ((j) >= n0 ? k + ((size_t)((j)-n0) * Hkv + (g)) * d \
                               : c->Kr + ((size_t)(g) * w + (size_t)((j) % w)) * d)
#define TOK_V(j, g) ((j) >= n0 ? v + ((size_t)((j)-n0) * Hkv + (g)) * d \
                               : c->Vr + ((size_t)(g) * w + (size_t)((j) % w)) * d)

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
      phi_softmax(qt, d, phiq);
      /* in the state before the call started */
      const double *S = c->S + (size_t)g * d * d;
      const double *z = c->z + (size_t)g * d;
      double denl = 0.0;
      for (int col = 0; col < d; ++col) numl[col] = 0.0;
      for (int r = 0; r < d; ++r) {
        denl += phiq[r] * z[r];
        for (int col = 0; col < d; ++col) numl[col] += phiq[r] * S[(size_t)r * d + col];
      }
      /* entered the state since the call started: tokens max(0, n0-delay) .. t-delay, explicit */
      int64_t e_lo = n0 - delay;
      if (e_lo < 0) e_lo = 0;
      for (int64_t j = e_lo; j <= t - delay; ++j) {
        phi_softmax(TOK_K(j, g), d, phik);
        double c_j = dot(phiq, phik, d);
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
    for (int64_t j = e_lo; j < n1 - delay; ++j) fold(c, g, TOK_K(j, g), TOK_V(j, g), phik);
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
      }
  }
#undef TOK_K
#undef TOK_V
  c->n = n1;
  free(phiq);
  free(phik);
  free(num);
  free(numl);
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

/* Copies of the state: ringK, ringV [Hkv][w][d]; S [Hkv][d][d]; z [Hkv][d]. Any may be NULL. */
void glide_oracle_cell_export(const glide_oracle_cell *c, double *ringK, double *ringV,
                              double *S, double *z) {
  size_t ring = (size_t)c->Hkv * (size_t)c->w * c->d;
  if (ringK && ring) memcpy(ringK, c->Kr, ring * sizeof(double));
  if (ringV && ring) memcpy(ringV, c->Vr, ring * sizeof(double));
  if (S) memcpy(S, c->S, (size_t)c->Hkv * c->d * c->d * sizeof(double));
  if (z) memcpy(z, c->z, (size_t)c->Hkv * c->d * sizeof(double));
}

int glide_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
