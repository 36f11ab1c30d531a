/*
 * Reference oracle for the Sentinel verifier check (arXiv 2603.03592) -- TEST INFRASTRUCTURE.
 * See sentinel_oracle.h.  Plain C, float64, one explicit loop per definition.
 */
#include "sentinel_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------ */
/* element helpers                                                                       */

double so_bf16(uint16_t bits) {
  uint32_t u = (uint32_t)bits << 16; /* bf16 is the upper half of an IEEE binary32 */
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

uint16_t so_bf16_round(double v) {
  if (isnan(v)) return 0x7FC0;
  const uint16_t sign = signbit(v) ? 0x8000 : 0x0000;
  const double a = fabs(v);
  if (isinf(a)) return (uint16_t)(sign | 0x7F80);
  /* lo = the largest bf16 magnitude <= a, hi = the next one; pick the nearer, ties to even */
  float f = (float)a;
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  u &= 0xFFFF0000u;
  if (so_bf16((uint16_t)(u >> 16)) > a) u -= 0x10000u;   /* the float rounding went above a */
  const uint16_t lo = (uint16_t)(u >> 16), hi = (uint16_t)(lo + 1);
  const double dlo = a - so_bf16(lo);
  /* past the largest finite bf16 the next grid point is 2^128, which rounds to infinity */
  const double dhi = (isinf(so_bf16(hi)) ? ldexp(1.0, 128) : so_bf16(hi)) - a;
  uint16_t pick;
  if (dlo < dhi) pick = lo;
  else if (dlo > dhi) pick = hi;
  else pick = (lo & 1) ? hi : lo;
  return (uint16_t)(sign | pick);
}

/* three-valued sign: -1, 0, +1 (both zeros give 0) */
static int sign3(double v) { return (v > 0.0) - (v < 0.0); }

void so_default_params(so_params *p) {
  memset(p, 0, sizeof *p);
  /* Tab. "verification_config", column "8x16 Mesh, 0.6B": activation | gradient */
  p->beta[0] = 0.90;     p->beta[1] = 0.80;
  p->k0[0] = 1.5;        p->k0[1] = 3.0;
  p->alpha[0] = 1e-4;    p->alpha[1] = 1e-3;
  p->n_max[0] = 10;      p->n_max[1] = 10;
  p->gamma_g[0] = 1.1;   p->gamma_g[1] = 1.01;
  p->gamma_s[0] = 0.9;   p->gamma_s[1] = 0.99;
  p->lambda[0] = 0.15;   p->lambda[1] = 0.05;
  p->eps[0] = 1e-3;      p->eps[1] = 5e-5;
  p->shrink_ratio = 0.5;
  p->severe_mult = 100.0;        /* Sec. 3.1, "Violation Counter with Forgiveness" */
  p->l = 100;                    /* Sec. 5: window of the past 100 steps            */
  p->c = 5;                      /* Sec. 3.1                                        */
  p->t_forgiveness = 100;        /* Sec. 3.1                                        */
  p->metric_mask = 15u;
  p->B = 1; p->T = 1; p->d = 8;
  p->R = 1;
  p->ema_bf16 = 0;
  p->ref_over_batch = 0;
  p->ref_over_tokens = 0;
}

/* ------------------------------------------------------------------------------------ */
/* Sec. 3.1: the distance measures Omega_i(x, m) of one unit                             */

int so_distance(const uint16_t *x, const double *m, size_t n, double gamma[3], double stat[8]) {
  size_t e;
  const double dn = (double)n;

  for (e = 0; e < n; ++e) {
    if (!isfinite(so_bf16(x[e]))) {
      int i;
      for (i = 0; i < 3; ++i) gamma[i] = NAN;
      for (i = 0; i < SO_NSTAT; ++i) stat[i] = NAN;
      return 1;
    }
  }

  /* Mean absolute difference: the average over all features of |x_e - m_e|. */
  double abs_sum = 0.0;
  for (e = 0; e < n; ++e) abs_sum += fabs(so_bf16(x[e]) - m[e]);
  gamma[SO_L1] = abs_sum / dn;

  /* Normalised Euclidean distance: z-score x and m (scalar mean and population standard
   * deviation over all elements of the unit), then average the squared difference.  A vector
   * whose elements are all equal has standard deviation 0 and z-scores to the zero vector. */
  double sum_x = 0.0, sum_m = 0.0;
  double min_x = so_bf16(x[0]), max_x = min_x, min_m = m[0], max_m = min_m;
  for (e = 0; e < n; ++e) {
    const double xe = so_bf16(x[e]), me = m[e];
    sum_x += xe; sum_m += me;
    if (xe < min_x) min_x = xe;
    if (xe > max_x) max_x = xe;
    if (me < min_m) min_m = me;
    if (me > max_m) max_m = me;
  }
  const double mu_x = sum_x / dn, mu_m = sum_m / dn;
  double ss_x = 0.0, ss_m = 0.0, ss_xm = 0.0, sq_x = 0.0, sq_m = 0.0;
  for (e = 0; e < n; ++e) {
    const double xe = so_bf16(x[e]), me = m[e];
    ss_x += (xe - mu_x) * (xe - mu_x);
    ss_m += (me - mu_m) * (me - mu_m);
    ss_xm += (xe - mu_x) * (me - mu_m);
    sq_x += xe * xe;
    sq_m += me * me;
  }
  const double var_x = (min_x == max_x) ? 0.0 : ss_x / dn;
  const double var_m = (min_m == max_m) ? 0.0 : ss_m / dn;
  const double sd_x = sqrt(var_x), sd_m = sqrt(var_m);
  double z_sum = 0.0;
  for (e = 0; e < n; ++e) {
    const double zx = (sd_x > 0.0) ? (so_bf16(x[e]) - mu_x) / sd_x : 0.0;
    const double zm = (sd_m > 0.0) ? (m[e] - mu_m) / sd_m : 0.0;
    z_sum += (zx - zm) * (zx - zm);
  }
  gamma[SO_L2Z] = z_sum / dn;

  /* Sign flip ratio: the fraction of coordinates whose signs differ. */
  size_t flips = 0;
  for (e = 0; e < n; ++e) flips += (sign3(so_bf16(x[e])) != sign3(m[e]));
  gamma[SO_SFR] = (double)flips / dn;

  stat[0] = mu_x; stat[1] = var_x; stat[2] = sqrt(sq_x);
  stat[3] = mu_m; stat[4] = var_m; stat[5] = ss_xm / dn; stat[6] = sqrt(sq_m);
  stat[7] = (sd_x > 0.0 && sd_m > 0.0) ? (ss_xm / dn) / (sd_x * sd_m) : 0.0;
  return 0;
}

/* ------------------------------------------------------------------------------------ */
/* Sec. 3.1: sliced Wasserstein distance                                                  */

static int cmp_double(const void *a, const void *b);

double so_sliced_wasserstein(const uint16_t *x, const double *m, size_t tokens, size_t d,
                             const uint16_t *u, size_t L, double *w1_per_direction) {
  size_t t, c, l;
  for (t = 0; t < tokens * d; ++t)
    if (!isfinite(so_bf16(x[t]))) return NAN;
  double *px = (double *)malloc(tokens * sizeof(double));
  double *pm = (double *)malloc(tokens * sizeof(double));
  double total = 0.0;
  for (l = 0; l < L; ++l) {
    /* push both clouds forward along direction u_l: one number per token */
    for (t = 0; t < tokens; ++t) {
      double ax = 0.0, am = 0.0;
      for (c = 0; c < d; ++c) {
        const double ul = so_bf16(u[l * d + c]);
        ax += so_bf16(x[t * d + c]) * ul;
        am += m[t * d + c] * ul;
      }
      px[t] = ax;
      pm[t] = am;
    }
    /* W1 of two empirical measures with equally many atoms: match the order statistics */
    qsort(px, tokens, sizeof(double), cmp_double);
    qsort(pm, tokens, sizeof(double), cmp_double);
    double w1 = 0.0;
    for (t = 0; t < tokens; ++t) w1 += fabs(px[t] - pm[t]);
    w1 /= (double)tokens;
    if (w1_per_direction) w1_per_direction[l] = w1;
    total += w1;
  }
  free(px); free(pm);
  return total / (double)L;
}

/* ------------------------------------------------------------------------------------ */
/* Alg. 5: adaptive IQR thresholds                                                       */

double so_percentile(const double *sorted, size_t n, double p) {
  const double pos = p * (double)(n - 1);
  const size_t lo = (size_t)floor(pos);
  const size_t hi = (lo + 1 < n) ? lo + 1 : lo;
  const double frac = pos - (double)lo;
  return sorted[lo] + frac * (sorted[hi] - sorted[lo]);
}

static int cmp_double(const void *a, const void *b) {
  const double x = *(const double *)a, y = *(const double *)b;
  return (x > y) - (x < y);
}

/* fraction of the window strictly outside the closed interval [lo, hi] */
static double fp_rate(const double *w, size_t n, double lo, double hi) {
  size_t out = 0, j;
  for (j = 0; j < n; ++j) out += (w[j] < lo || w[j] > hi);
  return (double)out / (double)n;
}

int so_adaptive_iqr(const double *window, size_t n, double alpha, int n_max, double gamma_g,
                    double gamma_s, double lambda, double eps, double shrink_ratio,
                    double thr[6], int iters[2]) {
  if (iters) { iters[0] = 0; iters[1] = 0; }
  if (n == 0) return 0;

  double *sorted = (double *)malloc(n * sizeof(double));
  memcpy(sorted, window, n * sizeof(double));
  qsort(sorted, n, sizeof(double), cmp_double);
  const double q1 = so_percentile(sorted, n, 0.25);
  const double q2 = so_percentile(sorted, n, 0.50);
  const double q3 = so_percentile(sorted, n, 0.75);
  free(sorted);

  const double iqr = fmax(q3 - q1, eps);
  double k = thr[3]; /* the multiplier persists from call to call */
  double tau_lower = q2 - k * iqr;
  double tau_upper = q2 + k * iqr;
  double fp = fp_rate(window, n, tau_lower, tau_upper);

  int it = 0;
  while (fp > alpha && it < n_max) { /* widen */
    k = k * gamma_g;
    tau_lower = q2 - k * iqr;
    tau_upper = q2 + k * iqr;
    fp = fp_rate(window, n, tau_lower, tau_upper);
    ++it;
  }
  if (iters) iters[0] = it;

  it = 0;
  while (fp < shrink_ratio * alpha && it < n_max) { /* narrow */
    k = k * gamma_s;
    tau_lower = q2 - k * iqr;
    tau_upper = q2 + k * iqr;
    fp = fp_rate(window, n, tau_lower, tau_upper);
    ++it;
  }
  if (iters) iters[1] = it;

  const double d_min = fabs(q2) * lambda; /* minimum distance from the median */
  tau_lower = fmin(tau_lower, q2 - d_min);
  tau_upper = fmax(tau_upper, q2 + d_min);

  thr[0] = q1; thr[1] = q2; thr[2] = q3; thr[3] = k; thr[4] = tau_lower; thr[5] = tau_upper;
  return 1;
}

/* ------------------------------------------------------------------------------------ */
/* verifier state                                                                        */

typedef struct so_window {      /* one history list, oldest first */
  double *v;
  size_t n, cap;
} so_window;

typedef struct so_kind_state {
  double *m;                                  /* EMA reference, B*T*d, starts at zero */
  so_window hist[2][SO_NMETRIC];              /* [level][metric]                      */
  double thr[2][SO_NMETRIC][SO_NTHR];
  int has_thr[2][SO_NMETRIC];
  double *stats;                              /* (1+B)*8 of the last call             */
  long steps;
  int last_flagged;                           /* the last verified step raised a flag */
} so_kind_state;

struct so_verifier {
  so_params p;
  size_t N, Ns, Nm;
  so_kind_state ks[2];
  int violations[SO_MAX_WORKERS], clean_streak[SO_MAX_WORKERS], banned[SO_MAX_WORKERS];
  uint16_t *u;   /* directions of the sliced Wasserstein metric, bf16 [n_dir][d]; NULL = metric off */
  int n_dir;
  int nm;        /* metrics in use: 3, or 4 once directions are set */
};

static void window_push(so_window *w, double val) {
  if (w->n == w->cap) { /* truncate to the last `cap` entries: the oldest leaves */
    memmove(w->v, w->v + 1, (w->cap - 1) * sizeof(double));
    w->n = w->cap - 1;
  }
  w->v[w->n++] = val;
}

/* which element of the reference stands for element e of a [B,T,d] tensor */
static size_t ref_index(const so_verifier *v, size_t e) {
  const size_t d = (size_t)v->p.d, c = e % d, t = (e / d) % (size_t)v->p.T, b = e / v->Ns;
  const size_t tt = v->p.ref_over_tokens ? 0 : t, bb = v->p.ref_over_batch ? 0 : b;
  const size_t rows_per_sample = v->p.ref_over_tokens ? 1 : (size_t)v->p.T;
  return (bb * rows_per_sample + tt) * d + c;
}

so_verifier *so_create(const so_params *p) {
  if (p->B < 1 || p->T < 1 || p->d < 1 || p->l < 1 || p->R < 1 || p->R > SO_MAX_WORKERS) return NULL;
  if (p->ref_over_batch && (p->R != 1 || p->ema_bf16)) return NULL;   /* likewise the [T,d] reference */
  if (p->ref_over_tokens && (p->R != 1 || p->ema_bf16)) return NULL;  /* and the [B,d] / [d] references */
  so_verifier *v = (so_verifier *)calloc(1, sizeof *v);
  v->p = *p;
  v->Ns = (size_t)p->T * (size_t)p->d;
  v->N = v->Ns * (size_t)p->B;
  /* elements of the reference: [B,T,d], [T,d] (over the samples), [B,d] (over the tokens), [d] (over both) */
  v->Nm = (p->ref_over_batch ? 1u : (size_t)p->B) * (p->ref_over_tokens ? 1u : (size_t)p->T) * (size_t)p->d;
  v->u = NULL; v->n_dir = 0; v->nm = 3;
  for (int kind = 0; kind < 2; ++kind) {
    so_kind_state *ks = &v->ks[kind];
    ks->m = (double *)calloc(v->Nm, sizeof(double));
    ks->stats = (double *)calloc((size_t)(1 + p->B) * SO_NSTAT, sizeof(double));
    for (int L = 0; L < 2; ++L)
      for (int i = 0; i < SO_NMETRIC; ++i) {
        so_window *w = &ks->hist[L][i];
        /* the window spans l iterations of all R workers (and of their B samples) */
        w->cap = (size_t)p->l * (size_t)p->R * ((L == 0) ? 1u : (size_t)p->B);
        w->v = (double *)calloc(w->cap, sizeof(double));
        w->n = 0;
        ks->thr[L][i][3] = p->k0[kind];
        ks->has_thr[L][i] = 0;
      }
  }
  return v;
}

int so_set_directions(so_verifier *v, const uint16_t *u, int n_dir) {
  if (n_dir < 1 || !u || v->p.ref_over_batch) return -1;
  if (v->ks[0].steps || v->ks[1].steps) return -1;   /* the metric set is fixed before the first step */
  free(v->u);
  v->u = (uint16_t *)malloc((size_t)n_dir * (size_t)v->p.d * sizeof(uint16_t));
  memcpy(v->u, u, (size_t)n_dir * (size_t)v->p.d * sizeof(uint16_t));
  v->n_dir = n_dir;
  v->nm = SO_NMETRIC;
  return 0;
}

void so_destroy(so_verifier *v) {
  if (!v) return;
  for (int kind = 0; kind < 2; ++kind) {
    free(v->ks[kind].m);
    free(v->ks[kind].stats);
    for (int L = 0; L < 2; ++L)
      for (int i = 0; i < SO_NMETRIC; ++i) free(v->ks[kind].hist[L][i].v);
  }
  free(v->u);
  free(v);
}

/* scores and statistics of every unit against the current EMA: row 0 = the whole tensor,
 * row 1+b = sample b.  Returns a bit per row set when that row holds non-finite input. */
static void all_units(so_verifier *v, const uint16_t *x, int kind, double *gam, int *nonfinite) {
  so_kind_state *ks = &v->ks[kind];
  const size_t d = (size_t)v->p.d;
  /* a [T,d] reference stands for the same tensor in every sample, a [d] reference for the same
   * vector in every token: write the broadcast out */
  double *wide = NULL;
  if (v->Nm != v->N) {
    wide = (double *)malloc(v->N * sizeof(double));
    for (size_t e = 0; e < v->N; ++e) wide[e] = ks->m[ref_index(v, e)];
  }
  const double *m = wide ? wide : ks->m;
  for (int r = 0; r <= v->p.B; ++r) {
    /* unit r: the whole tensor (B*T tokens) or sample r-1 (T tokens) */
    const size_t off = (r == 0) ? 0 : (size_t)(r - 1) * v->Ns;
    const size_t n = (r == 0) ? v->N : v->Ns;
    double *g = gam + (size_t)r * SO_NMETRIC;
    nonfinite[r] = so_distance(x + off, m + off, n, g, ks->stats + (size_t)r * SO_NSTAT);
    g[SO_SW] = v->u ? so_sliced_wasserstein(x + off, m + off, n / d, d, v->u, (size_t)v->n_dir, NULL)
                    : NAN;
  }
  free(wide);
}

static void refresh_thresholds(so_verifier *v, int kind) {
  so_kind_state *ks = &v->ks[kind];
  const so_params *p = &v->p;
  for (int L = 0; L < 2; ++L)
    for (int i = 0; i < v->nm; ++i) {
      so_window *w = &ks->hist[L][i];
      if (so_adaptive_iqr(w->v, w->n, p->alpha[kind], p->n_max[kind], p->gamma_g[kind],
                          p->gamma_s[kind], p->lambda[kind], p->eps[kind], p->shrink_ratio,
                          ks->thr[L][i], NULL))
        ks->has_thr[L][i] = 1;
    }
}

/* Eq. (1) with one submission per update (the per-trainer form of the SWARM appendix). */
static void ema_update(so_verifier *v, const uint16_t *x, int kind) {
  double *m = v->ks[kind].m;
  const double beta = v->p.beta[kind];
  if (v->p.ema_bf16) {
    /* The reference is stored as bf16.  Which of two neighbouring bf16 values an element takes
     * is a decision of the arithmetic, so it is taken in the arithmetic of the stored format's
     * producer: single precision, one fused multiply-add, then one rounding to nearest even. */
    const float bf = (float)beta, of = (float)(1.0 - beta);
    for (size_t e = 0; e < v->N; ++e)
      m[e] = so_bf16(so_bf16_round((double)fmaf(bf, (float)m[e], of * (float)so_bf16(x[e]))));
    return;
  }
  if (v->Nm != v->N) {   /* Eq. 1 with the mean over the samples and / or tokens as the submission */
    const size_t copies = v->N / v->Nm;
    double *sum = (double *)calloc(v->Nm, sizeof(double));
    for (size_t e = 0; e < v->N; ++e) sum[ref_index(v, e)] += so_bf16(x[e]);
    for (size_t i = 0; i < v->Nm; ++i) m[i] = beta * m[i] + (1.0 - beta) * (sum[i] / (double)copies);
    free(sum);
    return;
  }
  for (size_t e = 0; e < v->N; ++e) m[e] = beta * m[e] + (1.0 - beta) * so_bf16(x[e]);
}

/* Eq. 3 / Alg. 5: a deviation is out of bounds when it does not lie in the closed interval
 * [tau_lower, tau_upper].  Written as the negation of "lies inside", so that a deviation that is
 * not a number counts as outside (and, being flagged, never joins the history). */
int so_out_of_bounds(double gamma, double tau_lower, double tau_upper) {
  return !(gamma >= tau_lower && gamma <= tau_upper);
}

/* Sec. 3.1: a worker is banned at once when its deviation lies "x100 above the threshold".  The
 * rule speaks of a deviation that broke the threshold, so it is looked at only for a metric
 * that flagged: |gamma - q2| >= severe_mult * (tau_upper - q2). */
int so_severe(int flagged, double gamma, double q2, double tau_upper, double severe_mult) {
  return flagged && fabs(gamma - q2) >= severe_mult * (tau_upper - q2);
}

/* The first level of the reduction, for one token row: sum_c x, sum_c x^2, sum_c |x - m| and the
 * number of channels with sign(x) != sign(m) (Sec. 3.1 measures before the mean over tokens). */
void so_token_sums(const uint16_t *x, const double *m, size_t d, double out[4]) {
  out[0] = out[1] = out[2] = out[3] = 0.0;
  for (size_t c = 0; c < d; ++c) {
    const double xv = so_bf16(x[c]);
    out[0] += xv;
    out[1] += xv * xv;
    out[2] += fabs(xv - m[c]);
    out[3] += (sign3(xv) != sign3(m[c])) ? 1.0 : 0.0;
  }
}

/* Sec. 3.1, violation counter with forgiveness, kept per worker */
void so_count_violation(so_verifier *v, int r, int flagged, int severe) {
  const so_params *p = &v->p;
  if (flagged) {
    v->violations[r] += 1;
    v->clean_streak[r] = 0;
    if (v->violations[r] >= p->c || severe) v->banned[r] = 1;
  } else {
    v->clean_streak[r] += 1;
    if (v->clean_streak[r] >= p->t_forgiveness) {
      v->violations[r] = (v->violations[r] > 0) ? v->violations[r] - 1 : 0;
      v->clean_streak[r] = 0;
    }
  }
}

int so_update_reference(so_verifier *v, const uint16_t *x, int kind, double *scores) {
  const int rows = 1 + v->p.B;
  so_kind_state *ks = &v->ks[kind];
  double *gam = (double *)malloc((size_t)rows * SO_NMETRIC * sizeof(double));
  int *nf = (int *)malloc((size_t)rows * sizeof(int));
  all_units(v, x, kind, gam, nf);
  if (scores) memcpy(scores, gam, (size_t)rows * SO_NMETRIC * sizeof(double));
  ks->steps += 1;
  const int bad = nf[0];
  if (!bad) {
    /* warm-up: every deviation joins the history, then thresholds, then the EMA */
    for (int i = 0; i < v->nm; ++i) window_push(&ks->hist[0][i], gam[i]);
    for (int b = 0; b < v->p.B; ++b)
      for (int i = 0; i < v->nm; ++i)
        window_push(&ks->hist[1][i], gam[(size_t)(1 + b) * SO_NMETRIC + i]);
    refresh_thresholds(v, kind);
    ema_update(v, x, kind);
  }
  free(gam); free(nf);
  return bad;
}

int so_verify(so_verifier *v, const uint16_t *x, int kind, double *scores, uint32_t *flags) {
  const so_params *p = &v->p;
  const int rows = 1 + p->B;
  so_kind_state *ks = &v->ks[kind];
  double *gam = (double *)malloc((size_t)rows * SO_NMETRIC * sizeof(double));
  int *nf = (int *)malloc((size_t)rows * sizeof(int));

  /* 1. Gamma_i = Omega_i(x_t, m_{t-1}) for every unit */
  all_units(v, x, kind, gam, nf);
  memcpy(scores, gam, (size_t)rows * SO_NMETRIC * sizeof(double));
  ks->steps += 1;

  /* 2. Tukey test against the thresholds left by the previous step */
  int any_flag = 0, severe = 0, no_thr = 0;
  for (int r = 0; r < rows; ++r) {
    const int L = (r == 0) ? 0 : 1;
    uint32_t f = 0;
    if (nf[r]) {
      f |= SO_FLAG_NONFINITE;
    } else {
      for (int i = 0; i < v->nm; ++i) {
        if (!ks->has_thr[L][i]) { no_thr = 1; continue; }
        if (!((p->metric_mask >> i) & 1u)) continue;
        const double *t = ks->thr[L][i];
        const double g = gam[(size_t)r * SO_NMETRIC + i];
        const int out = so_out_of_bounds(g, t[4], t[5]);
        if (out) f |= (1u << i);
        /* 3. severe deviation, tested on the whole-tensor unit */
        if (r == 0 && so_severe(out, g, t[1], t[5], p->severe_mult)) severe = 1;
      }
    }
    flags[r] = f;
    if (f) any_flag = 1;
  }

  /* 4. violation counter with forgiveness */
  so_count_violation(v, 0, any_flag, severe);

  /* 5. clean units join the history; thresholds are refreshed for the next step */
  for (int r = 0; r < rows; ++r) {
    if (flags[r]) continue;
    const int L = (r == 0) ? 0 : 1;
    for (int i = 0; i < v->nm; ++i)
      window_push(&ks->hist[L][i], gam[(size_t)r * SO_NMETRIC + i]);
  }
  refresh_thresholds(v, kind);

  /* 6. the EMA moves only when nothing was flagged */
  const int commit = !any_flag;
  ks->last_flagged = any_flag;
  if (commit) ema_update(v, x, kind);

  if (commit) flags[0] |= SO_FLAG_COMMITTED;
  if (severe) flags[0] |= SO_FLAG_SEVERE;
  if (v->banned[0]) flags[0] |= SO_FLAG_BANNED;
  if (no_thr) flags[0] |= SO_FLAG_NO_THRESHOLDS;
  free(gam); free(nf);
  return commit;
}

void so_worker_counters(const so_verifier *v, int r, int out[3]) {
  out[0] = v->violations[r]; out[1] = v->clean_streak[r]; out[2] = v->banned[r];
}

int so_step_replicas(so_verifier *v, const uint16_t *const *xs, int kind, int warmup,
                     unsigned tainted_in, double *scores, uint32_t *flags) {
  const so_params *p = &v->p;
  const int R = p->R, rows = 1 + p->B;
  so_kind_state *ks = &v->ks[kind];
  double *gam = (double *)malloc((size_t)rows * SO_NMETRIC * sizeof(double));
  int *nf = (int *)malloc((size_t)rows * sizeof(int));
  int collected[SO_MAX_WORKERS], tainted[SO_MAX_WORKERS], severe_w[SO_MAX_WORKERS];
  int elsewhere[SO_MAX_WORKERS];            /* tainted at another stage: not collected here */
  int no_thr = 0;
  ks->steps += 1;
  if (warmup) tainted_in = 0;               /* the warm-up phase has honest workers only */

  for (int r = 0; r < R; ++r) {
    double *sc = scores + (size_t)r * rows * SO_NMETRIC;
    uint32_t *fl = flags + (size_t)r * rows;
    collected[r] = 0; tainted[r] = 0; severe_w[r] = 0; elsewhere[r] = 0;
    for (int u = 0; u < rows; ++u) fl[u] = 0;
    if (!warmup && v->banned[r]) {          /* banned workers are not collected any more */
      for (int j = 0; j < rows * SO_NMETRIC; ++j) sc[j] = NAN;
      continue;
    }
    if ((tainted_in >> r) & 1u) {
      /* Alg. 3: a worker tainted at another stage is marked and not collected; Alg. 2 leaves
       * such a worker out of its loop.  Either way: no metrics, no counter, no history. */
      for (int j = 0; j < rows * SO_NMETRIC; ++j) sc[j] = NAN;
      elsewhere[r] = 1;
      continue;
    }
    collected[r] = 1;
    all_units(v, xs[r], kind, gam, nf);     /* Gamma = Omega(x_t^(r), m_{t-1}) */
    memcpy(sc, gam, (size_t)rows * SO_NMETRIC * sizeof(double));
    int any_flag = 0;
    for (int u = 0; u < rows; ++u) {
      const int L = (u == 0) ? 0 : 1;
      uint32_t f = 0;
      if (nf[u]) {
        f |= SO_FLAG_NONFINITE;
      } else if (!warmup) {
        for (int i = 0; i < v->nm; ++i) {
          if (!ks->has_thr[L][i]) { no_thr = 1; continue; }
          if (!((p->metric_mask >> i) & 1u)) continue;
          const double *t = ks->thr[L][i];
          const double g = gam[(size_t)u * SO_NMETRIC + i];
          const int out = so_out_of_bounds(g, t[4], t[5]);
          if (out) f |= (1u << i);
          if (u == 0 && so_severe(out, g, t[1], t[5], p->severe_mult)) severe_w[r] = 1;
        }
      }
      fl[u] = f;
      if (f) any_flag = 1;
    }
    tainted[r] = any_flag;
    if (!warmup) so_count_violation(v, r, any_flag, severe_w[r]);
    /* deviations of unflagged units join the pooled history (warm-up: of every unit, unless
     * the submission is non-finite) */
    if (!(warmup && any_flag))
      for (int u = 0; u < rows; ++u) {
        if (fl[u]) continue;
        const int L = (u == 0) ? 0 : 1;
        for (int i = 0; i < v->nm; ++i)
          window_push(&ks->hist[L][i], gam[(size_t)u * SO_NMETRIC + i]);
      }
  }
  refresh_thresholds(v, kind);              /* once, after the worker loop */

  /* more than half of the workers still in the pool flagged: a natural shift, not an attack */
  int n_tainted = 0, n_banned = 0, n_elsewhere = 0, natural = 0;
  for (int r = 0; r < R; ++r) { n_tainted += tainted[r]; n_banned += v->banned[r]; n_elsewhere += elsewhere[r]; }
  /* the stage's tainted set: the workers flagged here and, for gradients (Alg. 3), the ones
   * marked as tainted at another stage */
  const int n_stage = n_tainted + (kind == SO_GRAD ? n_elsewhere : 0);
  if (!warmup && 2 * n_stage > R - n_banned) {
    natural = 1;
    for (int r = 0; r < R; ++r)
      if (!(flags[(size_t)r * rows] & SO_FLAG_NONFINITE)) tainted[r] = 0;
  }

  /* Eq. 1 with the mean over the clean submissions */
  int n_clean = 0;
  for (int r = 0; r < R; ++r) n_clean += (collected[r] && !tainted[r]);
  if (n_clean > 0) {
    double *m = ks->m;
    const double beta = p->beta[kind];
    if (p->ema_bf16) {
      /* The reference is stored as bf16: as for one submission per update, which of two
       * neighbouring bf16 values an element takes is decided in single precision -- the clean
       * submissions added up in worker order, weighted by (1-beta)/|clean|, one fused
       * multiply-add with beta m, one rounding to nearest even. */
      const float bf = (float)beta, wf = (float)(1.0 - beta) / (float)n_clean;
      for (size_t e = 0; e < v->N; ++e) {
        float sum = 0.0f;
        for (int r = 0; r < R; ++r)
          if (collected[r] && !tainted[r]) sum += (float)so_bf16(xs[r][e]);
        m[e] = so_bf16(so_bf16_round((double)fmaf(bf, (float)m[e], wf * sum)));
      }
    } else
    for (size_t e = 0; e < v->N; ++e) {
      double sum = 0.0;
      for (int r = 0; r < R; ++r)
        if (collected[r] && !tainted[r]) sum += so_bf16(xs[r][e]);
      m[e] = beta * m[e] + (1.0 - beta) * (sum / (double)n_clean);
    }
  }
  ks->last_flagged = (n_stage > 0) && !natural;
  for (int r = 0; r < R; ++r) {
    uint32_t *fl = flags + (size_t)r * rows;
    if (collected[r] && !tainted[r]) fl[0] |= SO_FLAG_COMMITTED;
    if (severe_w[r]) fl[0] |= SO_FLAG_SEVERE;
    if (!warmup && v->banned[r]) fl[0] |= SO_FLAG_BANNED;
    if (no_thr && collected[r]) fl[0] |= SO_FLAG_NO_THRESHOLDS;
    if (natural) fl[0] |= SO_FLAG_NATURAL_SHIFT;
    if (elsewhere[r]) fl[0] |= SO_FLAG_TAINTED_ELSEWHERE;
  }
  free(gam); free(nf);
  return n_clean;
}

int so_replace_if_flagged(const so_verifier *v, uint16_t *x, int kind, int fill) {
  if (!v->ks[kind].last_flagged) return 0;
  const double *m = v->ks[kind].m;                 /* a flagged step left m at m_{t-1} */
  for (size_t e = 0; e < v->N; ++e) x[e] = fill ? 0 : so_bf16_round(m[ref_index(v, e)]);
  return 1;
}

void so_skip_tainted(so_verifier *v, int kind) {
  v->ks[kind].steps += 1;
  v->ks[kind].last_flagged = 1;
}

void so_reset_worker(so_verifier *v) {
  for (int r = 0; r < SO_MAX_WORKERS; ++r) { v->violations[r] = 0; v->clean_streak[r] = 0; v->banned[r] = 0; }
}

/* ------------------------------------------------------------------------------------ */
/* accessors                                                                             */

const double *so_ema(const so_verifier *v, int kind) { return v->ks[kind].m; }

void so_set_ema(so_verifier *v, int kind, const double *m) {
  memcpy(v->ks[kind].m, m, v->Nm * sizeof(double));
  if (v->p.ema_bf16)
    for (size_t e = 0; e < v->N; ++e) v->ks[kind].m[e] = so_bf16(so_bf16_round(m[e]));
}

size_t so_history(const so_verifier *v, int kind, int level, int metric, double *out, size_t cap) {
  const so_window *w = &v->ks[kind].hist[level][metric];
  const size_t n = (w->n < cap) ? w->n : cap;
  if (out) memcpy(out, w->v, n * sizeof(double));
  return w->n;
}

int so_thresholds(const so_verifier *v, int kind, int level, int metric, double thr[6]) {
  memcpy(thr, v->ks[kind].thr[level][metric], SO_NTHR * sizeof(double));
  return v->ks[kind].has_thr[level][metric];
}

void so_last_stats(const so_verifier *v, int kind, double *stats) {
  memcpy(stats, v->ks[kind].stats, (size_t)(1 + v->p.B) * SO_NSTAT * sizeof(double));
}

void so_counters(const so_verifier *v, int out[3]) {
  out[0] = v->violations[0]; out[1] = v->clean_streak[0]; out[2] = v->banned[0];
}

long so_steps(const so_verifier *v, int kind) { return v->ks[kind].steps; }
