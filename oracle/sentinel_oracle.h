/*
 * Reference oracle for the Sentinel verifier check (arXiv 2603.03592).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 CPU restatement of what the
 * paper defines: the distance measures of Sec. 3.1, the EMA reference of Eq. (1) in its
 * one-submission-per-update (SWARM trainer) form, the per-submission body of Alg. 2 / Alg. 3,
 * the warm-up body of Alg. 1 and the adaptive IQR thresholds of Alg. 5.  It exists so that
 * tests can check the CUDA library against it and so that the benchmark can time it as a
 * reported CPU baseline.  It shares no code with the CUDA library and must never be linked,
 * imported or called from the product path.
 *
 * Every metric is written from its definition (two passes for the z-scores, an explicit
 * loop per element); nothing is blocked, fused or reordered.
 *
 * Parity unpinned (the paper gives no value to pin these conventions to; each is a
 * parameter so that a later correction is one constant):
 *   - the meaning of "FP-rate << alpha" in Alg. 5 (read as FP-rate < shrink_ratio * alpha),
 *   - the "x100 above the threshold" severe-deviation rule of Sec. 3.1,
 *   - the forgiveness bookkeeping ("decrements after T_forgiveness consecutive clean steps"),
 *   - the percentile convention (linear interpolation at p*(n-1)).
 *   - how a worker tainted at another stage enters this stage's bookkeeping (Alg. 2 leaves it
 *     out of its loop, Alg. 3 adds it to the stage's tainted set: read literally, per kind; a
 *     worker that was not collected never enters the mean of Eq. 1),
 *   - the number and the draw of the sliced Wasserstein directions (the caller supplies them),
 *   - the two storage variants the paper does not mention: a reference stored as bf16 (the one
 *     place where this oracle leaves float64: which of two neighbouring bf16 values an element
 *     takes is a decision of the arithmetic, so the update m = bf16(fma(beta, m, (1-beta) x)) is
 *     taken in single precision, the precision the stored format implies, and agrees with a
 *     single-precision implementation bit for bit; it is pinned to an independent float64
 *     emulation of that fused update, the choice of the variant itself is not the paper's), and the references reduced over the samples ([T,d]),
 *     over the tokens ([B,d]) or over both ([d]) (Eq. 1 with the mean over what is reduced).
 */
#ifndef SENTINEL_ORACLE_H
#define SENTINEL_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { SO_ACT = 0, SO_GRAD = 1 };                 /* h (forward) or g (backward)           */
enum { SO_L1 = 0, SO_L2Z = 1, SO_SFR = 2, SO_SW = 3, SO_NMETRIC = 4 };
enum { SO_NSTAT = 8 };                            /* mean_x var_x |x|_2 mean_m var_m cov |m|_2 rho */
enum { SO_MAX_WORKERS = 16 };
enum { SO_NTHR = 6 };                             /* q1 q2 q3 k tau_lower tau_upper        */

/* report bits, one word per unit (row 0 = whole tensor, rows 1..B = samples) */
enum {
  SO_FLAG_L1 = 1u << 0, SO_FLAG_L2Z = 1u << 1, SO_FLAG_SFR = 1u << 2, SO_FLAG_SW = 1u << 3,
  SO_FLAG_NONFINITE = 1u << 7,
  SO_FLAG_COMMITTED = 1u << 16, SO_FLAG_SEVERE = 1u << 17,
  SO_FLAG_BANNED = 1u << 18, SO_FLAG_NO_THRESHOLDS = 1u << 19,
  SO_FLAG_NATURAL_SHIFT = 1u << 20,  /* more than half of the workers flagged: taint cleared */
  SO_FLAG_TAINTED_ELSEWHERE = 1u << 21 /* the worker was tainted at another stage: not collected */
};

/* Hyper-parameters; index 0 = activations, 1 = gradients (Tab. "verification_config"). */
typedef struct so_params {
  double beta[2];          /* EMA decay, Eq. (1)                                   */
  double k0[2];            /* initial IQR multiplier, Alg. 5                        */
  double alpha[2];         /* target false-positive rate, Alg. 5                    */
  int    n_max[2];         /* max grow / shrink iterations, Alg. 5                  */
  double gamma_g[2];       /* grow factor  > 1                                      */
  double gamma_s[2];       /* shrink factor < 1                                     */
  double lambda[2];        /* minimum-distance multiplier                           */
  double eps[2];           /* IQR floor                                             */
  double shrink_ratio;     /* "FP-rate << alpha"  :=  FP-rate < shrink_ratio*alpha  */
  double severe_mult;      /* immediate ban when deviation >= severe_mult * allowed */
  int    l;                /* history window, in steps                              */
  int    c;                /* violations before a ban                               */
  int    t_forgiveness;    /* clean steps before the counter decrements             */
  unsigned metric_mask;    /* which metrics may raise a flag (bit i = metric i)     */
  int    B, T, d;          /* submission shape                                      */
  int    R;                /* workers (replicas) feeding this boundary, d_s >= 1    */
  int    ema_bf16;         /* != 0: the reference is stored as bf16                 */
  int    ref_over_batch;   /* != 0: one [T,d] reference for all B samples (R = 1)   */
  int    ref_over_tokens;  /* != 0: one reference row for all T tokens of a sample: [B,d], or
                              [d] together with ref_over_batch (R = 1)               */
} so_params;

typedef struct so_verifier so_verifier;

/* Defaults: the "8x16 mesh, 0.6B" column of the hyper-parameter table; c, T_forgiveness
 * from Sec. 3.1; l from Sec. 5. */
void so_default_params(so_params *p);

/* bf16 bit pattern -> double, exactly. */
double so_bf16(uint16_t bits);

/* Sec. 3.1 distance measures of one unit: n elements of x (bf16 bits) against n reference
 * values m.  gamma[3] = {L1, normalised L2, SFR}; stat[8] as listed above.  Returns 1 when x
 * holds a NaN or an infinity (then every output is NaN), else 0. */
int so_distance(const uint16_t *x, const double *m, size_t n, double gamma[3], double stat[8]);

/* The first reduction level for one token row of d channels: out = {sum_c x, sum_c x^2,
 * sum_c |x - m|, #{c : sign(x) != sign(m)}} (the per-token terms of the Sec. 3.1 measures). */
void so_token_sums(const uint16_t *x, const double *m, size_t d, double out[4]);

/* Eq. 3 / Alg. 5: 1 when gamma does not lie in [tau_lower, tau_upper]; a gamma that is not a
 * number is outside. */
int so_out_of_bounds(double gamma, double tau_lower, double tau_upper);

/* Sec. 3.1, immediate ban: 1 when the metric flagged and |gamma - q2| >= severe_mult *
 * (tau_upper - q2).  (Parity unpinned: the paper only says "x100 above the threshold".) */
int so_severe(int flagged, double gamma, double q2, double tau_upper, double severe_mult);

/* Percentile of an ascending array by linear interpolation at position p*(n-1), p in [0,1]. */
double so_percentile(const double *sorted, size_t n, double p);

/* Alg. 5 for one (kind, level, metric) window.  thr[SO_NTHR] holds q1 q2 q3 k tau_lower
 * tau_upper; on entry thr[3] is the multiplier carried over from the previous call (k0 the
 * first time).  An empty window leaves thr untouched and returns 0; otherwise returns 1.
 * iters[2], if not NULL, receives the number of grow and shrink iterations taken. */
int so_adaptive_iqr(const double *window, size_t n, double alpha, int n_max, double gamma_g,
                    double gamma_s, double lambda, double eps, double shrink_ratio,
                    double thr[6], int iters[2]);

so_verifier *so_create(const so_params *p);

/* Sec. 3.1: adds the sliced Wasserstein distance to the metric set M of this verifier.  u: the
 * caller's n_dir unit directions as bf16 bit patterns, [n_dir][d] (copied).  From then on every
 * unit's fourth score is so_sliced_wasserstein of the unit (B*T tokens for the whole tensor,
 * T tokens for a sample) against the EMA, with its own history and thresholds like the other
 * metrics; without directions the fourth score is NaN and takes no part.  Only before the
 * first step; returns 0, or -1 if refused. */
int so_set_directions(so_verifier *v, const uint16_t *u, int n_dir);
void so_destroy(so_verifier *v);

/* Warm-up step (Alg. 1, warm-up loop): scores against the current EMA, every unit appended
 * to the history, thresholds refreshed, EMA updated.  scores: (1+B)*4 doubles or NULL.
 * Returns 0, or 1 if the input was non-finite (then nothing changes). */
int so_update_reference(so_verifier *v, const uint16_t *x, int kind, double *scores);

/* Verified step (body of Alg. 2 / Alg. 3 for one submission).  scores: (1+B)*4 doubles,
 * flags: (1+B) words.  Returns 1 if the EMA was updated (no unit flagged), else 0. */
int so_verify(so_verifier *v, const uint16_t *x, int kind, double *scores, uint32_t *flags);

/* Sec. 3.1, sliced Wasserstein distance of one unit.  x (bf16 bits) and m are clouds of
 * `tokens` points in R^d (row-major [tokens][d]); u holds L directions as bf16 bit patterns,
 * [L][d], which the caller has normalised.  For every direction both clouds are projected, the
 * two sets of `tokens` projections are sorted, and W1 between the two empirical distributions
 * is the mean absolute difference of the order statistics; the result is the mean over the
 * L directions (a Monte-Carlo estimate of the expectation over the sphere with the caller's
 * draws).  w1_per_direction, if not NULL, receives the L terms.  Returns NaN if x holds a
 * non-finite value. */
double so_sliced_wasserstein(const uint16_t *x, const double *m, size_t tokens, size_t d,
                             const uint16_t *u, size_t L, double *w1_per_direction);

/* double -> bf16 bit pattern, round to nearest, ties to even (one rounding, straight from
 * the double). */
uint16_t so_bf16_round(double v);

/* Alg. 4 (GradientReplacement) for one submission: if the last verified step of `kind` was
 * flagged, x (n = B*T*d bf16 bit patterns) becomes the reference m_{t-1} rounded to bf16
 * (fill = 0) or zeros (fill = 1); otherwise x is left alone.  Returns 1 if it replaced. */
int so_replace_if_flagged(const so_verifier *v, uint16_t *x, int kind, int fill);

/* One iteration at this boundary with all R workers' submissions (Alg. 1 main loop, Alg. 2 /
 * Alg. 3 with their worker loop; the EMA is Eq. 1 with the mean over the clean workers).
 * xs[r] = worker r's tensor.  Every non-banned worker is scored against the same m_{t-1} and
 * tested against the same bounds; its violation counter, forgiveness and ban are its own;
 * clean units join the history pooled over workers (l*R entries at the tensor level, l*R*B at
 * the sample level); Alg. 5 runs once after the loop; if more than half of the non-banned
 * workers were flagged the taint set is cleared (natural distribution shift); the EMA moves
 * with the mean of the submissions that are not tainted.  warmup != 0: the warm-up loop of
 * Alg. 1 instead (no test, no counters, everything joins, mean over all workers).
 * tainted_in: bit r set = worker r was tainted at another stage in this iteration (Sec. 3.1,
 * cascading effects; the set "tainted downstream" of Alg. 3, the workers "in T_t" that the loop
 * of Alg. 2 leaves out).  Such a worker is not collected (xs[r] may be NULL): no metrics (NaN
 * scores), no counter change, no history entry, never part of the mean; its row 0 reports
 * SO_FLAG_TAINTED_ELSEWHERE.  For gradients it belongs to the stage's tainted set (Alg. 3) and
 * so counts towards the >50% rule and marks the step as flagged for Alg. 4; for activations it
 * does not (Alg. 2).  Ignored during warm-up; a banned worker is skipped as banned.
 * scores: [R][1+B][4]; flags: [R][1+B] (row 0 of each worker carries its status bits).
 * Returns the number of submissions that entered the EMA. */
int so_step_replicas(so_verifier *v, const uint16_t *const *xs, int kind, int warmup,
                     unsigned tainted_in, double *scores, uint32_t *flags);

/* The single-submission form of the same event: the one worker this verifier follows was
 * tainted at another stage in this step.  Nothing is collected or recorded; the step counts,
 * and it is marked flagged so that so_replace_if_flagged replaces the outgoing tensor. */
void so_skip_tainted(so_verifier *v, int kind);
void so_worker_counters(const so_verifier *v, int r, int out[3]);   /* v_r, streak, banned */
/* Sec. 3.1, "Violation Counter with Forgiveness", one step of worker r's counter: a violation
 * adds one and bans at c violations or on a severe deviation; T_forgiveness clean steps in a row
 * take one off.  (so_verify and so_step_replicas call this; it is exported so that a caller who
 * verifies the two kinds of a boundary in two oracle instances can keep their common counter.) */
void so_count_violation(so_verifier *v, int r, int flagged, int severe);

/* A new worker now feeds this boundary: clear its violation counter, streak and ban. */
void so_reset_worker(so_verifier *v);

/* State access for tests. */
const double *so_ema(const so_verifier *v, int kind);                 /* B*T*d values; T*d with ref_over_batch, B*d with ref_over_tokens, d with both */
void   so_set_ema(so_verifier *v, int kind, const double *m);
size_t so_history(const so_verifier *v, int kind, int level, int metric,
                  double *out, size_t cap);                            /* oldest first      */
int    so_thresholds(const so_verifier *v, int kind, int level, int metric, double thr[6]);
void   so_last_stats(const so_verifier *v, int kind, double *stats);  /* (1+B)*8           */
void   so_counters(const so_verifier *v, int out[3]);                 /* v, streak, banned */
long   so_steps(const so_verifier *v, int kind);

#ifdef __cplusplus
}
#endif
#endif
