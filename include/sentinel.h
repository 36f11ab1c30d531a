/*
 * libsentinel -- the verifier-node check of Sentinel (arXiv 2603.03592) for NVIDIA B200.
 *
 * A verifier sits between two pipeline stages and screens every tensor that crosses the
 * boundary: activations h on the way forward, activation-gradients g on the way back
 * (Sec. 2.1, Def. 2.1).  For each submitted tensor x it measures the distance to an
 * exponential moving average m of past clean submissions (Eq. 1, Eq. 2), compares each
 * distance with adaptive median/IQR bounds (Eq. 3, Alg. 5), reports flags, and moves the
 * average only when nothing was flagged.  One handle holds the state of one boundary for one
 * stream of submissions (the per-trainer form of the SWARM appendix: one tensor per update).
 *
 * Units.  Every quantity is computed for 1+B "units": row 0 is the whole tensor (the paper's
 * per-worker test), rows 1..B are the B samples, each tested on its own [T,d] slice against
 * the same slice of m with a history pooled over samples.
 *
 * Metrics (Sec. 3.1), index i:   0  L1    mean over elements of |x - m|
 *                                1  L2z   mean squared difference of the z-scored x and m
 *                                         (scalar mean / population std over the unit; a
 *                                         constant vector z-scores to zero)
 *                                2  SFR   fraction of elements with sign(x) != sign(m),
 *                                         sign in {-1,0,+1}
 *                                3  SW    sliced Wasserstein distance of the token clouds; only
 *                                         after sentinel_set_directions (else three metrics)
 *
 * Variants of a handle (sentinel_config): n_workers > 1 follows all workers of a stage and takes
 * their tensors together (the fixed-mesh form of Eq. 1, worker loop of Alg. 2 / Alg. 3);
 * ema_bf16 stores the reference as bf16; ref_over_batch keeps one [T,d] reference for all
 * samples, ref_over_tokens one vector per sample for all its tokens ([B,d]; with both: one [d]
 * vector).
 *
 * Conventions.  All tensors are dense, row-major [B,T,d] with d fastest (the _strided entry
 * points take padded rows).  x is bf16; the reference m is fp32 unless ema_bf16 is set, and is
 * owned by the library.  Pointers named dev_* are device pointers on
 * the handle's device, host_* are host pointers.  `cuda_stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  Calls only enqueue work unless stated otherwise;
 * outputs are valid once the stream reaches that point.  A handle is not thread-safe and its
 * calls must be stream-ordered; different handles are independent.
 *
 * Errors.  Every call returns 0 or a negative sentinel_status; nothing throws or aborts.
 * Arguments are checked before anything is launched, so an invalid call leaves the state
 * untouched.  sentinel_last_error() gives a message for the last failure.
 */
#ifndef SENTINEL_H
#define SENTINEL_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SENTINEL_NUM_METRICS 3     /* L1, z-scored L2, sign-flip ratio: the metrics every verifier uses */
#define SENTINEL_MAX_METRICS 4     /* ... plus the sliced Wasserstein distance once directions are set  */
#define SENTINEL_NUM_STATS 8      /* mean_x var_x |x|_2 mean_m var_m cov_xm |m|_2 rho */
#define SENTINEL_NUM_THRESHOLDS 6 /* q1 q2 q3 k tau_lower tau_upper                   */
#define SENTINEL_MAX_B 64         /* samples per tensor                               */
#define SENTINEL_MAX_WORKERS 16   /* workers (replicas of the stage) per handle       */
#define SENTINEL_MAX_WINDOW 4096  /* window_steps * n_workers * (B + 1) must not exceed this */

typedef enum sentinel_status {
  SENTINEL_OK = 0,
  SENTINEL_ERR_INVALID_ARG = -1,    /* NULL pointer, bad kind, value out of range           */
  SENTINEL_ERR_SHAPE_MISMATCH = -2, /* B,T,d differ from the handle's                       */
  SENTINEL_ERR_UNALIGNED = -3,      /* pointer not 16-byte aligned, or d not a multiple of 8 */
  SENTINEL_ERR_CUDA = -4,           /* a CUDA runtime call failed (see sentinel_last_error)  */
  SENTINEL_ERR_STATE_SIZE = -5,     /* state buffer too small or of another shape/version    */
  SENTINEL_ERR_TIMEOUT = -6,        /* reserved: a bounded device-side wait gave up          */
  SENTINEL_ERR_UNSUPPORTED = -7     /* shape or window beyond the compiled limits            */
} sentinel_status;

typedef enum sentinel_kind { SENTINEL_ACT = 0, SENTINEL_GRAD = 1 } sentinel_kind;

/* Bits of a flags word.  Rows 0..B carry the per-unit bits; row 0 also carries the status. */
#define SENTINEL_FLAG_L1 (1u << 0)            /* metric i outside [tau_lower, tau_upper]     */
#define SENTINEL_FLAG_L2Z (1u << 1)
#define SENTINEL_FLAG_SFR (1u << 2)
#define SENTINEL_FLAG_SWD (1u << 3)           /* sliced Wasserstein distance (needs directions) */
#define SENTINEL_FLAG_NONFINITE (1u << 7)     /* the unit holds a NaN or an infinity         */
#define SENTINEL_FLAG_COMMITTED (1u << 16)    /* row 0: the reference was updated            */
#define SENTINEL_FLAG_SEVERE (1u << 17)       /* row 0: deviation >= severe_mult * allowed   */
#define SENTINEL_FLAG_BANNED (1u << 18)       /* row 0: sticky until sentinel_reset_worker   */
#define SENTINEL_FLAG_NO_THRESHOLDS (1u << 19) /* row 0: some history was still empty         */
#define SENTINEL_FLAG_TAINTED_ELSEWHERE (1u << 21) /* row 0: tainted at another stage, not collected */
#define SENTINEL_FLAG_NATURAL_SHIFT (1u << 20) /* row 0: more than half of the workers flagged */

/* Hyper-parameters.  Arrays are indexed by kind.  Defaults: table "verification_config",
 * column "8x16 Mesh, 0.6B"; c and T_forgiveness from Sec. 3.1; the window from Sec. 5. */
typedef struct sentinel_config {
  double beta[2];          /* EMA decay (Eq. 1), in [0,1)                      0.90  0.80  */
  double k0[2];            /* initial IQR multiplier (Alg. 5)                  1.5   3.0   */
  double alpha[2];         /* target false-positive rate                       1e-4  1e-3  */
  int    n_max[2];         /* max widen / narrow iterations                    10    10    */
  double gamma_grow[2];    /* widen factor  (> 1)                              1.1   1.01  */
  double gamma_shrink[2];  /* narrow factor (< 1)                              0.9   0.99  */
  double lambda_min[2];    /* bounds at least lambda*|median| from the median  0.15  0.05  */
  double iqr_eps[2];       /* floor of the IQR                                 1e-3  5e-5  */
  double shrink_ratio;     /* narrow while FP-rate < shrink_ratio*alpha        0.5         */
  double severe_mult;      /* immediate ban multiple (Sec. 3.1)                100         */
  int    window_steps;     /* history length l, in steps                       100         */
  int    ban_violations;   /* c                                                5           */
  int    forgiveness_steps;/* T_forgiveness                                    100         */
  unsigned metric_mask;    /* bit i set: metric i may raise a flag             15          */
  int    B, T, d;          /* shape of every submission; B <= SENTINEL_MAX_B; d % 8 == 0
                              unless only the _strided entry points are used              */
  int    device;           /* CUDA device ordinal                                           */
  int    n_workers;        /* workers d_s feeding this boundary (multi-worker calls)   1    */
  int    ema_bf16;         /* 1: the reference is stored as bf16 (see below)           0    */
  int    ref_over_batch;   /* 1: one [T,d] reference for all B samples (see below)     0    */
  int    ref_over_tokens;  /* 1: one reference row for all T tokens of a sample: [B,d],
                              or [d] together with ref_over_batch (see below)          0    */
} sentinel_config;

typedef struct sentinel_verifier sentinel_verifier; /* opaque: one stage boundary */

/* Fills *cfg with the defaults above; B = T = d = 0 and device = 0 are left for the caller. */
/* ema_bf16 = 1 keeps the reference as bf16 instead of fp32: a verified tensor then moves
 * 2 B (x) + 2 B (reference read) + 2 B (candidate written) = 6 B per element instead of 10, and
 * the state takes half the memory.  The paper does not fix the reference's precision; with bf16
 * the update is m_t = bf16(fma(beta, m_{t-1}, (1-beta) x)) in single precision with one
 * rounding to nearest even, so a reference stops moving once (1-beta)|x - m| falls below half
 * a bf16 ulp of m (it settles within 1/(2(1-beta)) ulps of a steady input).  Scores, bounds and
 * flags are computed exactly as with fp32, against the rounded reference.  With n_workers > 1
 * the mean over the clean workers is taken in single precision in worker order and enters the
 * same one-rounding update; with sentinel_set_directions the projections of the reference are
 * taken from the stored bf16 values every step (a rounded reference does not follow the linear
 * recursion), so the chain reads 2 + 2 B/element.  State blobs carry the reference as fp32
 * either way (widened exactly on export, rounded to nearest even on import). */
/* ref_over_batch = 1 keeps ONE reference of shape [T,d] for all B samples of a tensor instead of
 * a [B,T,d] one (the paper states the reference only as "the EMA of the signal"; this reading
 * treats the samples of a microbatch as draws of the same [T,d] signal): every sample is compared
 * with it, the whole-tensor unit with B copies of it, and Eq. 1 moves it with the mean over the
 * samples, m_t = beta m_{t-1} + (1-beta)/B sum_b x[b].  A verified tensor then moves 2 + 8/B bytes
 * per element and the state shrinks B-fold.  Restrictions: n_workers = 1, fp32 reference,
 * B <= 16, d a multiple of 8; no strided tensors, no sentinel_set_directions, no per-token buffer.
 * Gradient replacement writes the one reference into every sample.  State blobs carry T*d
 * reference values per kind and record the shape in the header. */
/* ref_over_batch = 1 together with ref_over_tokens = 1 reduces the reference over the tokens as
 * well: ONE vector of d channels for all B*T token rows of a tensor (the same reading taken one
 * step further: every token is a draw of one d-dimensional signal).  Every token row is compared
 * with it -- sample b against T copies, the whole tensor against B*T copies -- and Eq. 1 moves it
 * with the mean over the token rows, m_t = beta m_{t-1} + (1-beta)/(B*T) sum_{b,t} x[b,t,:].  Only
 * x is read, 2 bytes per element, and the state of a kind is two vectors.  A step is two launches
 * (the streaming pass, then a small one that writes the candidate from the column sums and, if
 * the step committed, makes it the reference); both are enqueued by the same call.  Restrictions:
 * n_workers = 1, fp32 reference, d a multiple of 8; no strided tensors, no
 * sentinel_set_directions, no per-token buffer.  Gradient replacement writes the vector into
 * every token.  State blobs carry d reference values per kind; the header's shape field is 2.
 * ref_over_tokens = 1 alone keeps one such vector PER SAMPLE, a [B,d] reference: the tokens of
 * sample b are compared with vector b, which Eq. 1 moves with the mean over that sample's T token
 * rows; everything else as above.  State blobs then carry B*d values per kind, shape field 3. */
int sentinel_default_config(sentinel_config *cfg);

/* Allocates the state of one boundary on cfg->device: two fp32 [B,T,d] buffers per kind (the
 * reference and its candidate; m_0 = 0 as in Alg. 1), the history windows, thresholds and
 * counters.  Synchronous.  The library owns this memory until sentinel_destroy. */
int sentinel_verifier_create(const sentinel_config *cfg, sentinel_verifier **out);

/* Verified step: the body of Alg. 2 (kind = ACT) / Alg. 3 (kind = GRAD) for one submission.
 *   Gamma_i = Omega_i(x, m_{t-1}) for every unit (Eq. 2); a unit is flagged when an enabled
 *   metric lies outside the bounds left by the previous step (Eq. 3, Alg. 5); any flag is one
 *   violation (counter, forgiveness, ban: Sec. 3.1); unflagged units join the history and the
 *   bounds are refreshed; m_t = beta m_{t-1} + (1-beta) x only if nothing was flagged.
 * dev_x          bf16 [B,T,d], 16-byte aligned, read once.
 * dev_scores_out fp32 [(1+B)*M], scores_out[row*M+i] = Gamma_i of that unit (NaN for a
 *                non-finite unit); M = sentinel_num_metrics(h): 3, or 4 once directions are set.
 * dev_flags_out  u32 [1+B], bits as defined above.
 * x is read exactly once; the library keeps no reference to caller memory afterwards. */
int sentinel_verify(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T,
                    int d, void *cuda_stream, float *dev_scores_out, unsigned *dev_flags_out);

/* Sec. 3.1: adds the sliced Wasserstein distance to this verifier's metric set.  From the next
 * step on every unit has a fourth score, SW(unit, m_{t-1}) as sentinel_sliced_wasserstein
 * defines it (B*T tokens for the whole tensor, T for a sample), with its own history window,
 * bounds and flag bit (SENTINEL_FLAG_SWD, metric_mask bit 3) like the other three; score
 * rows, sentinel_get_thresholds and the replica calls then carry M = 4 columns.
 * dev_u_bf16: bf16 [L, d] unit directions chosen by the caller (the paper fixes neither
 * their number nor their draw), 16-byte aligned; copied on cuda_stream, and the call waits
 * for it.  L must be 4, 8 or 16; L*d*2 bytes <= 200 KiB; T <= 16384; d a multiple of 8.
 * Every later step first runs the projection / sort launches on the caller's stream, then the
 * streaming launch, which picks the distances up.  With one submission per update the
 * projections of the reference are carried along from step to step (Eq. 1 is linear), so the
 * chain reads x once more (2 B/element) and not the reference; with n_workers > 1, with a
 * bf16 reference, and on the first step after sentinel_import_state, it reads the reference
 * too.  The projections are fp32: inputs whose
 * projections leave the fp32 range give a score that is not a number, which counts as a
 * flag.  Allowed only before the first step and before sentinel_import_state
 * (SENTINEL_ERR_INVALID_ARG afterwards); the four windows' working copies must fit the
 * 200 KiB of shared memory (about window_steps*n_workers*(B+1) <= 3000), else
 * SENTINEL_ERR_UNSUPPORTED.  The strided entry points refuse a verifier with directions.
 * The scratch (about 24*L*B*T bytes) belongs to the handle. */
int sentinel_set_directions(sentinel_verifier *h, const void *dev_u_bf16, int L, void *cuda_stream);

/* Metrics this verifier uses (M above): 3, or 4 after sentinel_set_directions; 0 if h is NULL. */
int sentinel_num_metrics(const sentinel_verifier *h);

/* Warm-up step (the warm-up loop of Alg. 1, honest workers only): scores as above, every unit
 * joins the history, the bounds are refreshed and the reference is updated unconditionally.
 * No flags, no counters.  A non-finite x changes nothing.  dev_scores_out may be NULL. */
int sentinel_update_reference(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B,
                              int T, int d, void *cuda_stream, float *dev_scores_out);

/* sentinel_verify / sentinel_update_reference for a tensor whose rows are not packed: row
 * (b,t) starts row_stride elements after the previous one (row_stride >= d) and dev_x needs
 * 2-byte alignment only; d may be any positive number.  This is the layout of a
 * subspace-compressed signal, of which the verifier checks x[:, :, :-1] (SWARM appendix,
 * "compatibility with subspace compression"): pass the [B,T,k+1] tensor with d = k and
 * row_stride = k+1.  The reference stays dense [B,T,d].  Same arithmetic.  With d a multiple
 * of 8 the 128/256-bit accesses are kept and x is read in aligned 16-byte words that are shifted
 * into place: bytes of such a word that lie outside the verified elements (up to 14 before the
 * first element of a row or after its last one) are read and ignored, and no word is read that
 * holds no verified element.  With any other d the accesses are scalar (slower).  A handle
 * created with d % 8 != 0 can only be used through these two calls (and the queries /
 * checkpointing). */
int sentinel_verify_strided(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T,
                            int d, long long row_stride, void *cuda_stream, float *dev_scores_out,
                            unsigned *dev_flags_out);
int sentinel_update_reference_strided(sentinel_verifier *h, const void *dev_x, sentinel_kind kind,
                                      int B, int T, int d, long long row_stride, void *cuda_stream,
                                      float *dev_scores_out);

/* sentinel_verify for callers whose tensor and results live in host memory: copies x to a
 * staging buffer owned by the handle (allocated on first use), runs the check, copies scores
 * and flags back and waits for the stream.  host_x: bf16 [B,T,d] (pinned memory copies
 * fastest); host_scores_out: fp32 [(1+B)*M]; host_flags_out: u32 [1+B]. */
int sentinel_verify_host(sentinel_verifier *h, const void *host_x, sentinel_kind kind, int B,
                         int T, int d, void *cuda_stream, float *host_scores_out,
                         unsigned *host_flags_out);

/* Stateless form of Eq. 2 / Sec. 3.1: the three distances and the statistics of x against a
 * reference supplied by the caller.  dev_m: fp32 [B,T,d], 16-byte aligned.  dev_scores_out
 * fp32 [(1+B)*3]; dev_stats_out fp32 [(1+B)*8] or NULL.  Needs a few KiB of scratch, which it
 * takes from and returns to the stream's memory pool (cudaMallocAsync).  On first use the
 * library raises the release threshold of the device's default pool to 64 MiB (never lowers
 * it), so that the scratch is not handed back to the driver at every synchronisation. */
int sentinel_distance(const void *dev_x, const float *dev_m, int B, int T, int d, int device,
                      void *cuda_stream, float *dev_scores_out, float *dev_stats_out);

/* Sliced Wasserstein distance (Sec. 3.1), stateless: x and the reference m are read as clouds
 * of tokens in R^d (B*T points for the whole tensor, T points for a sample); along each of L
 * directions both clouds are projected, W1 of the two sets of projections is the mean
 * absolute difference of their order statistics, and the L values are averaged.
 * dev_u_bf16: the directions, bf16 [L, d], unit vectors chosen by the caller (the paper fixes
 * neither their number nor their draw), 16-byte aligned.  L must be 4, 8 or 16; L*d*2 bytes
 * must fit in 200 KiB of shared memory; T <= 16384.  dev_m: fp32 [B,T,d].
 * dev_sw_out: fp32 [1+B], row 0 the whole tensor, row 1+b sample b; NaN propagates from a
 * non-finite x.  Scratch (the projections, about 24*L*B*T bytes) comes from and returns to
 * the stream's memory pool. */
int sentinel_sliced_wasserstein(const void *dev_x, const float *dev_m, const void *dev_u_bf16, int L,
                                int B, int T, int d, int device, void *cuda_stream,
                                float *dev_sw_out);

/* The same computation as sentinel_distance for callers that must not allocate device memory
 * while they run: code whose memory pool has been frozen after start-up, real-time loops
 * that cannot afford an allocator call of unbounded duration, and processes whose
 * device-memory budget was handed out up front and may not grow.  (The paper
 * has no counterpart; this is a property of the library, not of the method.)
 * The kernel's scratch (two 64-byte partial slots per streaming CTA plus a ticket word) lives
 * in a fixed array of SENTINEL_NOALLOC_SCRATCH_BYTES that is part of the library image, so
 * every GPU that loads the library holds those bytes until the process exits.  The call
 * performs no cudaMalloc / cudaFree / pool allocation of any kind; inputs and outputs are
 * still the caller's.  If this device's launch needs more scratch than the array holds the
 * call fails with SENTINEL_ERR_UNSUPPORTED and a message naming both sizes; nothing is
 * launched.
 * The first call on each device looks up the array's device address (once per device, under a
 * lock); make that first call outside any stream capture.  All calls on a device share the
 * one array: it keeps whatever the last call left, so each call re-zeroes its ticket word on
 * the stream before launching, and two calls whose kernels could overlap on the GPU (two
 * streams, two threads) race on it -- order them on one stream or with events. */
#define SENTINEL_NOALLOC_SCRATCH_BYTES 65536
int sentinel_distance_noalloc(const void *dev_x, const float *dev_m, int B, int T, int d,
                              int device, void *cuda_stream, float *dev_scores_out,
                              float *dev_stats_out);

/* Statistics of the last call of this kind, fp32 [(1+B)*8] per unit:
 * mean_x, var_x, ||x||_2, mean_m, var_m, cov(x,m), ||m||_2, Pearson rho.  Enqueues a copy. */
int sentinel_get_stats(sentinel_verifier *h, sentinel_kind kind, float *dev_stats_out,
                       void *cuda_stream);

/* Current bounds, host_out double [2 levels][M metrics][6] = q1 q2 q3 k tau_lower tau_upper
 * (level 0 = whole tensor, 1 = samples; M = sentinel_num_metrics(h)); host_valid int [2][M]
 * (0 while that history is empty), may be NULL.  Waits for the stream. */
int sentinel_get_thresholds(sentinel_verifier *h, sentinel_kind kind, double *host_out,
                            int *host_valid, void *cuda_stream);

/* host_out int64 [6]: violations v, clean streak, banned (of worker 0), steps(ACT),
 * steps(GRAD), the error word written by device code: 0 = none, SENTINEL_DEVICE_STAGING_TIMEOUT =
 * a staged copy of the multi-worker, [T,d]- or [d]-reference kernels did not arrive within two
 * seconds (the warp's remaining rows were left out: the step's results are not to be used),
 * SENTINEL_DEVICE_OUT_OF_BOUNDS = the checked build skipped an access that would have left its
 * buffer (see sentinel_bounds_violations).  Waits for the stream. */
#define SENTINEL_DEVICE_STAGING_TIMEOUT 1
#define SENTINEL_DEVICE_OUT_OF_BOUNDS 2
int sentinel_get_counters(sentinel_verifier *h, long long *host_out, void *cuda_stream);

/* The checked build of the library (libsentinel_checked.so: the same sources compiled with
 * -DSENTINEL_CHECK_BOUNDS; the paper has no counterpart) compares every global-memory index that
 * its kernels derive from the shape -- B, T, d, the row stride, the number of CTAs, the window
 * sizes -- with the extent of the buffer before the access; an access that would leave the buffer
 * is skipped and counted, nothing traps.  host_count receives the number of skipped accesses on
 * `device` since the library was loaded, host_first_site (may be NULL) a code for where the first
 * one happened (0 = none).  Synchronises the device.  The normal build does no such checks:
 * there the call sets both to 0 and returns SENTINEL_ERR_UNSUPPORTED. */
int sentinel_bounds_violations(int device, unsigned long long *host_count, int *host_first_site);

/* host_out int64 [3]: violations, clean streak, banned of worker `worker`.  Waits. */
int sentinel_get_worker_counters(sentinel_verifier *h, int worker, long long *host_out, void *cuda_stream);

/* Per-token partial sums of the pass, written by every later call while registered:
 * dev_buf fp32 [B,T,4] = sum_c x, sum_c x^2, sum_c |x-m|, count of sign mismatches over the
 * token's d channels.  NULL unregisters.  The buffer stays the caller's. */
int sentinel_set_token_stats_buffer(sentinel_verifier *h, float *dev_buf);

/* One iteration with the submissions of all n_workers workers of the stage (the worker loop
 * of Alg. 2 / Alg. 3 and the reference update of Alg. 1 / Eq. 1).  host_dev_xs: a HOST array of
 * n_workers device pointers, each bf16 [B,T,d], 16-byte aligned (read by the call itself; the
 * tensors are read on the stream).  Every worker that is not banned is scored against the same
 * m_{t-1} and tested against the same bounds; violation counter, forgiveness and ban are kept
 * per worker; unflagged units join histories pooled over the workers (window_steps*n_workers
 * entries for the whole-tensor unit, times B for samples); the bounds are refreshed once per
 * iteration; if more than half of the workers still in the pool were flagged, the taint set
 * is cleared (natural distribution shift, SENTINEL_FLAG_NATURAL_SHIFT) and the counters stay
 * as they moved; the reference then moves with the mean of the untainted submissions.  All
 * workers are scored by ONE launch that reads every tensor and the reference once and writes
 * the mean over all collected workers into the spare reference buffer (2*R + 8 bytes per
 * element); if nobody was flagged that buffer becomes the reference, else a second launch takes
 * the mean over the clean workers from the untouched m_{t-1} (reading those tensors again).  A
 * banned worker is not read: its scores are NaN and its row 0 reports SENTINEL_FLAG_BANNED.
 * The per-token buffer of sentinel_set_token_stats_buffer is not written by these calls.
 * dev_scores_out fp32 [n_workers][1+B][M]; dev_flags_out u32 [n_workers][1+B]; row 0 of worker
 * r carries COMMITTED iff its tensor entered the mean. */
int sentinel_verify_replicas(sentinel_verifier *h, const void *const *host_dev_xs, sentinel_kind kind,
                             int B, int T, int d, void *cuda_stream, float *dev_scores_out,
                             unsigned *dev_flags_out);

/* sentinel_verify_replicas with the cascading-effect input of Sec. 3.1: bit r of tainted_in
 * says that worker r was tainted at another stage in this iteration (the set "tainted
 * downstream" of Alg. 3; the workers already in T_t that the loop of Alg. 2 leaves out).  Such
 * a worker is not collected: host_dev_xs[r] is ignored (may be NULL), its scores are NaN, its
 * counter, the histories and the mean are untouched, and its row 0 reports
 * SENTINEL_FLAG_TAINTED_ELSEWHERE.  For kind = GRAD it belongs to the stage's tainted set
 * (Alg. 3): it counts towards the >50% rule and leaves the step marked as flagged for
 * sentinel_replace_if_flagged; for kind = ACT it does not (Alg. 2).  A banned worker is
 * reported as banned whatever its bit says.  Bits at or above n_workers are an error. */
int sentinel_verify_replicas_tainted(sentinel_verifier *h, const void *const *host_dev_xs,
                                     sentinel_kind kind, unsigned tainted_in, int B, int T, int d,
                                     void *cuda_stream, float *dev_scores_out, unsigned *dev_flags_out);

/* The single-submission form of the same event: the worker this verifier follows was tainted
 * at another stage in this step.  Nothing is read or recorded (statistics paused, Sec. 3.1);
 * the step counts, and it is left marked as flagged so that sentinel_replace_if_flagged
 * overwrites the outgoing tensor (Alg. 4).  Enqueued on cuda_stream. */
int sentinel_skip_tainted(sentinel_verifier *h, sentinel_kind kind, void *cuda_stream);

/* The warm-up loop of Alg. 1 with all workers: no test, no counters, every unit of every worker
 * joins the history, the reference moves with the mean over all workers.  Outputs as above
 * (dev_flags_out may be NULL). */
int sentinel_update_reference_replicas(sentinel_verifier *h, const void *const *host_dev_xs,
                                       sentinel_kind kind, int B, int T, int d, void *cuda_stream,
                                       float *dev_scores_out, unsigned *dev_flags_out);

/* Gradient replacement (Alg. 4) for the submission this handle sees.  If the last
 * sentinel_verify of `kind` raised a flag (the step was not committed), dev_x_inout -- the
 * tensor about to be forwarded, bf16 [B,T,d], 16-byte aligned -- is overwritten with the stored
 * reference m_{t-1} rounded to bf16 (fill = 0), or with zeros (fill = 1, the variant the SWARM
 * appendix prefers); if it was clean, the tensor is left as it is.  The decision is taken on
 * the device: the call only enqueues work and never waits for the verify call before it.
 * dev_replaced_out (u32, may be NULL) receives 1 if the tensor was overwritten, else 0. */
int sentinel_replace_if_flagged(sentinel_verifier *h, void *dev_x_inout, sentinel_kind kind, int B,
                                int T, int d, int fill, void *cuda_stream,
                                unsigned *dev_replaced_out);

/* Worker slot `worker` (0 for single-submission use) is now fed by a new worker: clears its
 * violation counter, clean streak and ban.  Enqueued on cuda_stream. */
int sentinel_reset_worker(sentinel_verifier *h, int worker, void *cuda_stream);

/* Checkpointing.  The state is one self-describing blob: a 64-byte header
 * {u64 magic, u32 version = 3, i32 B, T, d, window_steps, n_workers, n_metrics, ref_over_batch}, then
 * i32 violations[16], clean_streak[16], banned[16], then per kind {i64 steps; i32 count[2];
 * i32 valid[2][4]; f64 thr[2][4][6]; f64 history[level 0: 4][window_steps*n_workers],
 * [level 1: 4][window_steps*n_workers*B] (oldest first, zero-padded); f32 m[B*T*d] (m[T*d] with
 * ref_over_batch, header field 1; m[d] with ref_over_tokens as well, field 2; m[B*d] with
 * ref_over_tokens alone, field 3)}.  The
 * layout always has room for four metrics; with n_metrics = 3 the fourth slots are unused.
 * A blob goes back only into a verifier with the same n_metrics (the directions themselves
 * are not part of the state: set them before importing).  Export and import wait for the
 * stream. */
size_t sentinel_state_bytes(const sentinel_verifier *h);
int sentinel_export_state(sentinel_verifier *h, void *host_buf, size_t n, void *cuda_stream);
int sentinel_import_state(sentinel_verifier *h, const void *host_buf, size_t n, void *cuda_stream);

/* Message of the last failure on this handle (h == NULL: of the calling thread's last failed
 * call that had no handle).  The string is owned by the library. */
const char *sentinel_last_error(const sentinel_verifier *h);

/* Frees everything the handle owns.  Waits for the device to finish the handle's work. */
int sentinel_destroy(sentinel_verifier *h);

#ifdef __cplusplus
}
#endif
#endif /* SENTINEL_H */
