/*
 * CPU oracle for the top-2 Mixture-of-Experts layer with expert pruning and
 * dynamic expert skipping (arXiv 2402.14800).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes; the CUDA library is checked against it.  It shares no code
 * with the CUDA path and must never be called from it.
 *
 * Conventions
 *   - All tensors arrive as bf16 bit patterns (uint16_t), row-major:
 *       x[T][h], W_gate[E][h], W1[E][f][h], W3[E][f][h], W2[E][h][f].
 *   - Contractions (router logits, expert projections) accumulate in double,
 *     ascending index order.
 *   - Decisions (softmax, top-2, skip test, renormalisation) are taken in fp32,
 *     the precision the kernels decide in, so that both sides compare the same
 *     quantities; the logits are the double sums rounded once to fp32.
 *   - bf16 rounding points (round-to-nearest-even), as a bf16 model has them:
 *       R1  the SwiGLU activation a = silu(W1 x) * (W3 x) is stored as bf16;
 *       R2  the layer output y is stored as bf16;
 *       R3  (search only) each expert output E_e(x) is stored as bf16.
 *   - Ties in top-2 go to the lower original expert index.
 *
 * Pins (tests/test_oracle_*.py): dense all-experts-then-mask in numpy fp64,
 * closed form w~_e0 = 1/(1+exp(l_e1-l_e0)), zero loss for the full subset,
 * integer count of tokens a subset disturbs, chunk additivity of loss^2,
 * per-subset recomputation == all-experts-once, beta>1 == top-1,
 * z^ - z = w~_e1 (f_e0 - f_e1), median beta skips exactly half.
 * Absolute output values have no printed example in the paper: parity for them
 * is pinned by the dense numpy restatement only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_MAX_E 16

/* ------------------------------------------------------------------ bf16 */

static float bf16_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* round-to-nearest-even on the upper 16 bits; NaN stays NaN */
static uint16_t f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16(f); }
float oracle_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------- router */

/* Router logits of one token for every expert (Sec. 3.1: l = W_gate x),
 * double accumulation, rounded once to fp32. */
static void router_logits(const uint16_t *x, const uint16_t *Wg, int h, int E, float *l) {
  for (int e = 0; e < E; ++e) {
    double acc = 0.0;
    const uint16_t *w = Wg + (size_t)e * h;
    for (int i = 0; i < h; ++i) acc += (double)bf16_to_f32(x[i]) * (double)bf16_to_f32(w[i]);
    l[e] = (float)acc;
  }
}

/* One token's routing among the kept experts.
 *   Sec. 3.1: w = Softmax(l); e_0, e_1 = indices of the largest and second
 *   largest w; Eq. 1: w~_ej = w_ej / (w_e0 + w_e1).
 *   Sec. 3.2: pruned experts are removed together with their router rows, so
 *   the softmax runs over the kept experts only.
 *   Sec. 3.3: e_1 is skipped when w_e1 < beta * w_e0 (strict).
 *   App. A.2 (i = 1, k = 2): after a skip the output is renormalised over the
 *   survivors, i.e. w~_e0 = 1.
 * Softmax is strictly increasing, so the order of w is the order of l and the
 * top-2 is taken on the logits (ties -> lower index).  With p_e = exp(l_e - l_e0)
 * (the max-subtracted softmax numerators, p_e0 = 1) and w_e = p_e / sum_kept p,
 * the common denominator cancels in every later quantity:
 *   w_e1 / w_e0 = p_e1,  skip <=> p_e1 < beta * p_e0,  w~_ej = p_ej / (p_e0 + p_e1).
 * They are evaluated in that cancelled form, so a token whose top-2 survives a
 * pruning keeps bit-identical weights.
 * Outputs: idx[2] original expert ids; w[2] softmax weights of e0,e1;
 * wn[2] weights applied to the expert outputs; ratio = w_e1 / w_e0. */
static void route_token(const float *l, int E, uint32_t kept, float beta, int32_t *idx, float *w,
                        float *wn, float *ratio, uint8_t *skipped) {
  int e0 = -1, e1 = -1;
  for (int e = 0; e < E; ++e)
    if (((kept >> e) & 1u) && (e0 < 0 || l[e] > l[e0])) e0 = e;
  for (int e = 0; e < E; ++e)
    if (((kept >> e) & 1u) && e != e0 && (e1 < 0 || l[e] > l[e1])) e1 = e;
  float p[ORACLE_MAX_E];
  float s = 0.0f;
  for (int e = 0; e < E; ++e) {
    if ((kept >> e) & 1u) {
      p[e] = expf(l[e] - l[e0]);
      s += p[e];
    }
  }
  idx[0] = e0;
  idx[1] = e1;
  w[0] = p[e0] / s;
  w[1] = p[e1] / s;
  *ratio = p[e1] / p[e0];
  *skipped = (uint8_t)(p[e1] < beta * p[e0]);
  if (*skipped) {
    wn[0] = 1.0f;
    wn[1] = 0.0f;
  } else {
    float d = p[e0] + p[e1];
    wn[0] = p[e0] / d;
    wn[1] = p[e1] / d;
  }
}

static int popcount32(uint32_t v) {
  int c = 0;
  while (v) {
    c += (int)(v & 1u);
    v >>= 1;
  }
  return c;
}

/* Routing of T tokens.  logits[T][E] (fp32, all E experts, optional),
 * idx[T][2], w[T][2], wn[T][2], ratio[T], skipped[T] (each optional). */
int oracle_route(const uint16_t *x, const uint16_t *Wg, int T, int h, int E, uint32_t kept_mask,
                 float beta, float *logits, int32_t *idx, float *w, float *wn, float *ratio,
                 uint8_t *skipped) {
  if (E < 2 || E > ORACLE_MAX_E || popcount32(kept_mask & ((1u << E) - 1u)) < 2) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    float l[ORACLE_MAX_E];
    int32_t id[2];
    float wr[2], wnn[2], rt;
    uint8_t sk;
    router_logits(x + (size_t)t * h, Wg, h, E, l);
    route_token(l, E, kept_mask, beta, id, wr, wnn, &rt, &sk);
    if (logits) memcpy(logits + (size_t)t * E, l, sizeof(float) * (size_t)E);
    if (idx) { idx[2 * t] = id[0]; idx[2 * t + 1] = id[1]; }
    if (w) { w[2 * t] = wr[0]; w[2 * t + 1] = wr[1]; }
    if (wn) { wn[2 * t] = wnn[0]; wn[2 * t + 1] = wnn[1]; }
    if (ratio) ratio[t] = rt;
    if (skipped) skipped[t] = sk;
  }
  return 0;
}

/* ---------------------------------------------------------------- expert */

/* SwiGLU expert E_e(x) = W2 ( silu(W1 x) * (W3 x) ) for one token (Sec. 3.1
 * names the transformation; Mixtral's form, no bias).  The activation is
 * rounded to bf16 (R1).  out[h] is the unrounded double result. */
static void expert_ffn(const uint16_t *x, const uint16_t *W1e, const uint16_t *W3e,
                       const uint16_t *W2e, int h, int f, double *out, float *a /* [f] scratch */) {
  for (int j = 0; j < f; ++j) {
    const uint16_t *w1 = W1e + (size_t)j * h;
    const uint16_t *w3 = W3e + (size_t)j * h;
    double g = 0.0, u = 0.0;
    for (int i = 0; i < h; ++i) {
      double xi = (double)bf16_to_f32(x[i]);
      g += xi * (double)bf16_to_f32(w1[i]);
      u += xi * (double)bf16_to_f32(w3[i]);
    }
    double act = g / (1.0 + exp(-g)) * u;
    a[j] = bf16_to_f32(f32_to_bf16((float)act));
  }
  for (int i = 0; i < h; ++i) {
    const uint16_t *w2 = W2e + (size_t)i * f;
    double o = 0.0;
    for (int j = 0; j < f; ++j) o += (double)a[j] * (double)bf16_to_f32(w2[j]);
    out[i] = o;
  }
}

/* Yall[T][E][h] (double): every expert applied to every token.  Experts whose
 * bit in expert_mask is clear are left untouched.  round_bf16 != 0 applies R3. */
int oracle_all_experts(const uint16_t *x, const uint16_t *W1, const uint16_t *W3,
                       const uint16_t *W2, int T, int h, int f, int E, uint32_t expert_mask,
                       int round_bf16, double *Yall) {
  if (E < 1 || E > ORACLE_MAX_E) return -1;
  long n = (long)T * E;
#pragma omp parallel
  {
    float *a = (float *)malloc(sizeof(float) * (size_t)f);
#pragma omp for schedule(dynamic, 1)
    for (long q = 0; q < n; ++q) {
      int t = (int)(q / E), e = (int)(q % E);
      if (!((expert_mask >> e) & 1u)) continue;
      double *o = Yall + (size_t)q * h;
      expert_ffn(x + (size_t)t * h, W1 + (size_t)e * f * h, W3 + (size_t)e * f * h,
                 W2 + (size_t)e * h * f, h, f, o, a);
      if (round_bf16)
        for (int i = 0; i < h; ++i) o[i] = (double)bf16_to_f32(f32_to_bf16((float)o[i]));
    }
    free(a);
  }
  return 0;
}

/* Expert co-selection counts (App. A.1): counts[a][b] = number of tokens whose largest
 * routing weight is expert a and second largest expert b (all experts kept, no skipping).
 * The activation frequency of expert e, which the frequency-based pruning baseline of
 * Sec. 4.1 ranks by, is the sum of row e and column e. */
int oracle_coselection(const uint16_t *x, const uint16_t *Wg, int T, int h, int E, int64_t *counts) {
  if (E < 2 || E > ORACLE_MAX_E) return -1;
  for (int i = 0; i < E * E; ++i) counts[i] = 0;
  uint32_t full = (1u << E) - 1u;
  for (int t = 0; t < T; ++t) {
    float l[ORACLE_MAX_E], wr[2], wnn[2], rt;
    int32_t id[2];
    uint8_t sk;
    router_logits(x + (size_t)t * h, Wg, h, E, l);
    route_token(l, E, full, 0.0f, id, wr, wnn, &rt, &sk);
    counts[id[0] * E + id[1]] += 1;
  }
  return 0;
}

/* Frequency baseline: keep the r experts with the highest activation frequency
 * (ties to the lower index). */
uint32_t oracle_frequency_subset(const int64_t *counts, int E, int r) {
  int64_t freq[ORACLE_MAX_E];
  for (int e = 0; e < E; ++e) {
    freq[e] = 0;
    for (int b = 0; b < E; ++b) freq[e] += counts[e * E + b] + counts[b * E + e];
  }
  uint32_t mask = 0;
  for (int k = 0; k < r; ++k) {
    int best = -1;
    for (int e = 0; e < E; ++e)
      if (!((mask >> e) & 1u) && (best < 0 || freq[e] > freq[best])) best = e;
    mask |= 1u << best;
  }
  return mask;
}

/* --------------------------------------------------------------- forward */

/* Pruned + skipping MoE layer forward (Eq. 2 with the routing above):
 *   z = w~_e0 E_e0(x) + w~_e1 E_e1(x), slot 0 first; a skipped e_1 is not
 *   evaluated.  y = bf16(residual + z) (R2); residual may be NULL (= 0).
 * Optional outputs: z64[T][h] unrounded (without residual), idx, wn, ratio,
 * skipped as in oracle_route. */
int oracle_moe_forward(const uint16_t *x, const uint16_t *Wg, const uint16_t *W1,
                       const uint16_t *W3, const uint16_t *W2, int T, int h, int f, int E,
                       uint32_t kept_mask, float beta, const uint16_t *residual, uint16_t *y,
                       double *z64, int32_t *idx, float *wn, float *ratio, uint8_t *skipped) {
  if (E < 2 || E > ORACLE_MAX_E || popcount32(kept_mask & ((1u << E) - 1u)) < 2) return -1;
#pragma omp parallel
  {
    float *a = (float *)malloc(sizeof(float) * (size_t)f);
    double *o0 = (double *)malloc(sizeof(double) * (size_t)h);
    double *o1 = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 1)
    for (int t = 0; t < T; ++t) {
      const uint16_t *xt = x + (size_t)t * h;
      float l[ORACLE_MAX_E], wr[2], wnn[2], rt;
      int32_t id[2];
      uint8_t sk;
      router_logits(xt, Wg, h, E, l);
      route_token(l, E, kept_mask, beta, id, wr, wnn, &rt, &sk);
      expert_ffn(xt, W1 + (size_t)id[0] * f * h, W3 + (size_t)id[0] * f * h,
                 W2 + (size_t)id[0] * h * f, h, f, o0, a);
      if (!sk)
        expert_ffn(xt, W1 + (size_t)id[1] * f * h, W3 + (size_t)id[1] * f * h,
                   W2 + (size_t)id[1] * h * f, h, f, o1, a);
      for (int i = 0; i < h; ++i) {
        double z = (double)wnn[0] * o0[i];
        if (!sk) z += (double)wnn[1] * o1[i];
        if (z64) z64[(size_t)t * h + i] = z;
        if (y) {
          double r = residual ? (double)bf16_to_f32(residual[(size_t)t * h + i]) : 0.0;
          y[(size_t)t * h + i] = f32_to_bf16((float)(r + z));
        }
      }
      if (idx) { idx[2 * t] = id[0]; idx[2 * t + 1] = id[1]; }
      if (wn) { wn[2 * t] = wnn[0]; wn[2 * t + 1] = wnn[1]; }
      if (ratio) ratio[t] = rt;
      if (skipped) skipped[t] = sk;
    }
    free(a);
    free(o0);
    free(o1);
  }
  return 0;
}

/* D_t = || E_e0(x_t) - E_e1(x_t) ||_2 over the token's two selected (kept) experts, the
 * quantity App. A.2 observes to be concentrated and replaces by a constant D. */
int oracle_top2_distance(const uint16_t *x, const uint16_t *Wg, const uint16_t *W1,
                         const uint16_t *W3, const uint16_t *W2, int T, int h, int f, int E,
                         uint32_t kept_mask, double *dist) {
  if (E < 2 || E > ORACLE_MAX_E || popcount32(kept_mask & ((1u << E) - 1u)) < 2) return -1;
#pragma omp parallel
  {
    float *a = (float *)malloc(sizeof(float) * (size_t)f);
    double *o0 = (double *)malloc(sizeof(double) * (size_t)h);
    double *o1 = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 1)
    for (int t = 0; t < T; ++t) {
      const uint16_t *xt = x + (size_t)t * h;
      float l[ORACLE_MAX_E], wr[2], wnn[2], rt;
      int32_t id[2];
      uint8_t sk;
      router_logits(xt, Wg, h, E, l);
      route_token(l, E, kept_mask, 0.0f, id, wr, wnn, &rt, &sk);
      expert_ffn(xt, W1 + (size_t)id[0] * f * h, W3 + (size_t)id[0] * f * h, W2 + (size_t)id[0] * h * f,
                 h, f, o0, a);
      expert_ffn(xt, W1 + (size_t)id[1] * f * h, W3 + (size_t)id[1] * f * h, W2 + (size_t)id[1] * h * f,
                 h, f, o1, a);
      double s2 = 0.0;
      for (int i = 0; i < h; ++i) s2 += (o0[i] - o1[i]) * (o0[i] - o1[i]);
      dist[t] = sqrt(s2);
    }
    free(a);
    free(o0);
    free(o1);
  }
  return 0;
}

/* ------------------------------------------------------- top-k generalisation */

/* Routing of one token in the general top-k setting (App. A.2).  e_0..e_{k-1} are the kept
 * experts with the k largest routing weights (ties to the lower index), p_m = exp(l_em - l_e0)
 * their softmax numerators (the denominator cancels everywhere).  Dynamic skipping keeps the
 * top-i* experts with
 *     i* = min i in 1..k  such that  sum_{m=i+1..k} w_m <= beta * sum_{m=1..k} w_m
 * (the paper's 1-based m), and the output is renormalised over those i* experts.
 * fp32 order of the sums, the same on the CUDA side: the total over the k experts in
 * ascending m; the tails accumulated from the smallest weight upwards; the kept mass in
 * ascending m. */
static void route_token_topk(const float *l, int E, uint32_t kept, int k, float beta, int32_t *idx,
                             float *wn, int *n_active, float *tail_frac) {
  uint32_t left = kept;
  float p[ORACLE_MAX_E];
  for (int m = 0; m < k; ++m) {
    int best = -1;
    for (int e = 0; e < E; ++e)
      if (((left >> e) & 1u) && (best < 0 || l[e] > l[best])) best = e;
    idx[m] = best;
    left &= ~(1u << best);
    p[m] = expf(l[best] - l[idx[0]]);
  }
  float total = 0.0f;
  for (int m = 0; m < k; ++m) total += p[m];
  float tail[ORACLE_MAX_E + 1];
  tail[k] = 0.0f;
  for (int m = k - 1; m >= 1; --m) tail[m] = tail[m + 1] + p[m];
  int istar = k;
  for (int i = 1; i <= k; ++i)
    if (tail[i] <= beta * total) { istar = i; break; }
  float keep = 0.0f;
  for (int m = 0; m < istar; ++m) keep += p[m];
  for (int m = 0; m < k; ++m) wn[m] = m < istar ? p[m] / keep : 0.0f;
  *n_active = istar;
  if (tail_frac) *tail_frac = tail[istar] / total;
}

/* Layer forward with top-k routing and the generalised skipping rule above.
 * idx[T][k], wn[T][k] (0 for skipped experts), n_active[T]; z64/y as in oracle_moe_forward;
 * tail_frac[T] = skipped mass / total mass of the k selected (0 when nothing is skipped). */
int oracle_moe_forward_topk(const uint16_t *x, const uint16_t *Wg, const uint16_t *W1,
                            const uint16_t *W3, const uint16_t *W2, int T, int h, int f, int E,
                            uint32_t kept_mask, int k, float beta, uint16_t *y, double *z64,
                            int32_t *idx, float *wn, int32_t *n_active, float *tail_frac,
                            float *logits) {
  if (E < 2 || E > ORACLE_MAX_E || k < 1 || popcount32(kept_mask & ((1u << E) - 1u)) < k) return -1;
#pragma omp parallel
  {
    float *a = (float *)malloc(sizeof(float) * (size_t)f);
    double *o = (double *)malloc(sizeof(double) * (size_t)h);
    double *z = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 1)
    for (int t = 0; t < T; ++t) {
      const uint16_t *xt = x + (size_t)t * h;
      float l[ORACLE_MAX_E], w[ORACLE_MAX_E], tf;
      int32_t id[ORACLE_MAX_E];
      int na;
      router_logits(xt, Wg, h, E, l);
      route_token_topk(l, E, kept_mask, k, beta, id, w, &na, &tf);
      for (int i = 0; i < h; ++i) z[i] = 0.0;
      for (int m = 0; m < na; ++m) {
        expert_ffn(xt, W1 + (size_t)id[m] * f * h, W3 + (size_t)id[m] * f * h,
                   W2 + (size_t)id[m] * h * f, h, f, o, a);
        for (int i = 0; i < h; ++i) z[i] += (double)w[m] * o[i];
      }
      for (int i = 0; i < h; ++i) {
        if (z64) z64[(size_t)t * h + i] = z[i];
        if (y) y[(size_t)t * h + i] = f32_to_bf16((float)z[i]);
      }
      for (int m = 0; m < k; ++m) {
        if (idx) idx[(size_t)t * k + m] = id[m];
        if (wn) wn[(size_t)t * k + m] = w[m];
      }
      if (n_active) n_active[t] = na;
      if (tail_frac) tail_frac[t] = tf;
      if (logits) memcpy(logits + (size_t)t * E, l, sizeof(float) * (size_t)E);
    }
    free(a);
    free(o);
    free(z);
  }
  return 0;
}

/* ------------------------------------------------------------------ beta */

static int cmp_float(const void *a, const void *b) {
  float fa = *(const float *)a, fb = *(const float *)b;
  return (fa > fb) - (fa < fb);
}

/* beta = median over the calibration tokens of w_e1 / w_e0 (Sec. 3.3).  For an
 * even count the two middle values are averaged (in double), so that exactly
 * half of a tie-free batch falls strictly below beta. */
int oracle_beta_median(const float *ratio, int T, float *beta) {
  if (T < 1) return -1;
  float *s = (float *)malloc(sizeof(float) * (size_t)T);
  memcpy(s, ratio, sizeof(float) * (size_t)T);
  qsort(s, (size_t)T, sizeof(float), cmp_float);
  if (T & 1)
    *beta = s[T / 2];
  else
    *beta = (float)(((double)s[T / 2 - 1] + (double)s[T / 2]) * 0.5);
  free(s);
  return 0;
}

/* ---------------------------------------------------------------- search */

static long binom(int n, int k) {
  if (k < 0 || k > n) return 0;
  long r = 1;
  for (int i = 1; i <= k; ++i) r = r * (n - k + i) / i;
  return r;
}

long oracle_num_subsets(int E, int r) { return binom(E, r); }

/* The r-subsets of {0..E-1} as bitmasks, in lexicographic order of their
 * ascending index tuples. */
int oracle_enumerate_subsets(int E, int r, uint32_t *masks) {
  if (r < 1 || r > E || E > ORACLE_MAX_E) return -1;
  int c[ORACLE_MAX_E];
  for (int i = 0; i < r; ++i) c[i] = i;
  long n = 0;
  for (;;) {
    uint32_t m = 0;
    for (int i = 0; i < r; ++i) m |= 1u << c[i];
    masks[n++] = m;
    int i = r - 1;
    while (i >= 0 && c[i] == E - r + i) --i;
    if (i < 0) break;
    ++c[i];
    for (int j = i + 1; j < r; ++j) c[j] = c[j - 1] + 1;
  }
  return 0;
}

/* Layer-wise pruning search, literal form of Eq. 3: for every subset C with
 * |C| = r build the pruned layer (router rows of pruned experts removed),
 * re-run it on every calibration token and take the Frobenius norm of the
 * difference to the unpruned layer's output.  No skipping on either side.
 * Expert outputs carry R3; the weighted sums stay unrounded.
 *   losses[nC]        Frobenius norms, subset order as above
 *   loss_sq[nC]       their squares (optional)
 *   n_changed[nC]     tokens with a non-zero error (optional)
 *   best_subset       bitmask of the argmin (first minimum wins) */
int oracle_prune_search_bruteforce(const uint16_t *x, const uint16_t *Wg, const uint16_t *W1,
                                   const uint16_t *W3, const uint16_t *W2, int T, int h, int f,
                                   int E, int r, double *losses, double *loss_sq,
                                   int64_t *n_changed, uint32_t *best_subset) {
  if (E < 2 || E > ORACLE_MAX_E || r < 2 || r > E) return -1;
  long nC = binom(E, r);
  uint32_t *masks = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)nC);
  oracle_enumerate_subsets(E, r, masks);
  uint32_t full = (1u << E) - 1u;
  double *sq = (double *)calloc((size_t)nC, sizeof(double));
  int64_t *nz = (int64_t *)calloc((size_t)nC, sizeof(int64_t));
  /* per-token squared errors, reduced over tokens in ascending order afterwards */
  double *err = (double *)malloc(sizeof(double) * (size_t)T);
  for (long c = 0; c < nC; ++c) {
#pragma omp parallel
    {
      float *a = (float *)malloc(sizeof(float) * (size_t)f);
      double *o = (double *)malloc(sizeof(double) * (size_t)h);
      double *F = (double *)malloc(sizeof(double) * (size_t)h);
      double *Fp = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 1)
      for (int t = 0; t < T; ++t) {
        const uint16_t *xt = x + (size_t)t * h;
        float l[ORACLE_MAX_E];
        router_logits(xt, Wg, h, E, l);
        for (int pass = 0; pass < 2; ++pass) {
          uint32_t kept = pass ? masks[c] : full;
          double *dst = pass ? Fp : F;
          int32_t id[2];
          float wr[2], wnn[2], rt;
          uint8_t sk;
          route_token(l, E, kept, 0.0f, id, wr, wnn, &rt, &sk);
          for (int i = 0; i < h; ++i) dst[i] = 0.0;
          for (int s = 0; s < 2; ++s) {
            int e = id[s];
            expert_ffn(xt, W1 + (size_t)e * f * h, W3 + (size_t)e * f * h, W2 + (size_t)e * h * f,
                       h, f, o, a);
            for (int i = 0; i < h; ++i)
              dst[i] += (double)wnn[s] * (double)bf16_to_f32(f32_to_bf16((float)o[i]));
          }
        }
        double e2 = 0.0;
        for (int i = 0; i < h; ++i) {
          double d = Fp[i] - F[i];
          e2 += d * d;
        }
        err[t] = e2;
      }
      free(a);
      free(o);
      free(F);
      free(Fp);
    }
    for (int t = 0; t < T; ++t) {
      sq[c] += err[t];
      nz[c] += (err[t] != 0.0);
    }
  }
  long best = 0;
  for (long c = 0; c < nC; ++c) {
    losses[c] = sqrt(sq[c]);
    if (loss_sq) loss_sq[c] = sq[c];
    if (n_changed) n_changed[c] = nz[c];
    if (losses[c] < losses[best]) best = c;
  }
  if (best_subset) *best_subset = masks[best];
  free(masks);
  free(sq);
  free(nz);
  free(err);
  return 0;
}

/* The same search with the experts evaluated once: Yall[t][e] = bf16(E_e(x_t))
 * for every (t, e), then each subset only re-routes among its kept logits and
 * gathers.  Must agree with the literal form above. */
int oracle_prune_search_allexperts(const uint16_t *x, const uint16_t *Wg, const uint16_t *W1,
                                   const uint16_t *W3, const uint16_t *W2, int T, int h, int f,
                                   int E, int r, double *losses, double *loss_sq,
                                   int64_t *n_changed, uint32_t *best_subset) {
  if (E < 2 || E > ORACLE_MAX_E || r < 2 || r > E) return -1;
  long nC = binom(E, r);
  uint32_t *masks = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)nC);
  oracle_enumerate_subsets(E, r, masks);
  uint32_t full = (1u << E) - 1u;
  double *Yall = (double *)malloc(sizeof(double) * (size_t)T * E * h);
  if (!Yall) { free(masks); return -2; }
  oracle_all_experts(x, W1, W3, W2, T, h, f, E, full, 1, Yall);
  double *err = (double *)malloc(sizeof(double) * (size_t)T * nC);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    float l[ORACLE_MAX_E];
    router_logits(x + (size_t)t * h, Wg, h, E, l);
    int32_t id[2], idc[2];
    float wr[2], wnF[2], wnC[2], rt;
    uint8_t sk;
    route_token(l, E, full, 0.0f, id, wr, wnF, &rt, &sk);
    const double *Y = Yall + (size_t)t * E * h;
    for (long c = 0; c < nC; ++c) {
      route_token(l, E, masks[c], 0.0f, idc, wr, wnC, &rt, &sk);
      double e2 = 0.0;
      for (int i = 0; i < h; ++i) {
        double F = (double)wnF[0] * Y[(size_t)id[0] * h + i] + (double)wnF[1] * Y[(size_t)id[1] * h + i];
        double Fp = (double)wnC[0] * Y[(size_t)idc[0] * h + i] + (double)wnC[1] * Y[(size_t)idc[1] * h + i];
        double d = Fp - F;
        e2 += d * d;
      }
      err[(size_t)t * nC + c] = e2;
    }
  }
  long best = 0;
  for (long c = 0; c < nC; ++c) {
    double sq = 0.0;
    int64_t nz = 0;
    for (int t = 0; t < T; ++t) {
      sq += err[(size_t)t * nC + c];
      nz += (err[(size_t)t * nC + c] != 0.0);
    }
    losses[c] = sqrt(sq);
    if (loss_sq) loss_sq[c] = sq;
    if (n_changed) n_changed[c] = nz;
  }
  for (long c = 0; c < nC; ++c)
    if (losses[c] < losses[best]) best = c;
  if (best_subset) *best_subset = masks[best];
  free(masks);
  free(Yall);
  free(err);
  return 0;
}

/* Progressive variant of the search (the "progressive" row of the paper's ablation on
 * layer-wise vs progressive pruning): the pruned layer is evaluated on x_p, the calibration
 * states that already went through the pruned earlier layers, while the target stays the
 * unpruned model's cached output F_ref[T][h] of this layer:
 *   loss(C) = || F'(x_p, C) - F_ref ||_F.
 * Expert outputs carry R3 as in the layer-wise search. */
int oracle_prune_search_progressive(const uint16_t *x_p, const uint16_t *Wg, const uint16_t *W1,
                                    const uint16_t *W3, const uint16_t *W2, const float *F_ref,
                                    int T, int h, int f, int E, int r, double *losses,
                                    double *loss_sq, uint32_t *best_subset) {
  if (E < 2 || E > ORACLE_MAX_E || r < 2 || r > E) return -1;
  long nC = binom(E, r);
  uint32_t *masks = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)nC);
  oracle_enumerate_subsets(E, r, masks);
  uint32_t full = (1u << E) - 1u;
  double *Yall = (double *)malloc(sizeof(double) * (size_t)T * E * h);
  if (!Yall) { free(masks); return -2; }
  oracle_all_experts(x_p, W1, W3, W2, T, h, f, E, full, 1, Yall);
  double *err = (double *)malloc(sizeof(double) * (size_t)T * nC);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    float l[ORACLE_MAX_E];
    router_logits(x_p + (size_t)t * h, Wg, h, E, l);
    int32_t idc[2];
    float wr[2], wnC[2], rt;
    uint8_t sk;
    const double *Y = Yall + (size_t)t * E * h;
    for (long c = 0; c < nC; ++c) {
      route_token(l, E, masks[c], 0.0f, idc, wr, wnC, &rt, &sk);
      double e2 = 0.0;
      for (int i = 0; i < h; ++i) {
        double Fp = (double)wnC[0] * Y[(size_t)idc[0] * h + i] + (double)wnC[1] * Y[(size_t)idc[1] * h + i];
        double d = Fp - (double)F_ref[(size_t)t * h + i];
        e2 += d * d;
      }
      err[(size_t)t * nC + c] = e2;
    }
  }
  long best = 0;
  for (long c = 0; c < nC; ++c) {
    double sq = 0.0;
    for (int t = 0; t < T; ++t) sq += err[(size_t)t * nC + c];
    losses[c] = sqrt(sq);
    if (loss_sq) loss_sq[c] = sq;
  }
  for (long c = 0; c < nC; ++c)
    if (losses[c] < losses[best]) best = c;
  if (best_subset) *best_subset = masks[best];
  free(masks);
  free(Yall);
  free(err);
  return 0;
}

/* ------------------------------------------------------------ stack glue */

/* RMSNorm with unit gain: out = bf16( x / sqrt(mean(x^2) + eps) ), as placed
 * before each MoE layer of the stacked workload. */
int oracle_rmsnorm(const uint16_t *x, int T, int h, double eps, uint16_t *out) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const uint16_t *xt = x + (size_t)t * h;
    double ss = 0.0;
    for (int i = 0; i < h; ++i) {
      double v = (double)bf16_to_f32(xt[i]);
      ss += v * v;
    }
    double inv = 1.0 / sqrt(ss / (double)h + eps);
    for (int i = 0; i < h; ++i)
      out[(size_t)t * h + i] = f32_to_bf16((float)((double)bf16_to_f32(xt[i]) * inv));
  }
  return 0;
}
