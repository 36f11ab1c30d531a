// Host side of libsentinel: argument checks, state ownership, launches.  See include/sentinel.h.
#include "sentinel.h"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "sentinel_kernels.cuh"
#include "sentinel_swd.cuh"

using namespace sentinel;

namespace {

thread_local std::string g_error;   // failures of calls that have no handle

constexpr unsigned long long kMagic = 0x4c454e49544e4553ull;  // "SENTINEL", little endian
constexpr unsigned kVersion = 3;
constexpr size_t kHeaderBytes = 64;

struct BlobHeader {
  unsigned long long magic;
  unsigned version;
  int B, T, d, window_steps, n_workers, n_metrics, ref_over_batch;
};

struct BlobWorkers {      // follows the header
  int violations[kMaxWorkers], clean_streak[kMaxWorkers], banned[kMaxWorkers];
};
static_assert(sizeof(BlobHeader) <= kHeaderBytes, "header must fit its slot");

struct BlobKindHead {
  long long steps;
  int count[2];
  int valid[2][kNumMetrics];
  double thr[2][kNumMetrics][kNumThr];
};
static_assert(sizeof(BlobKindHead) == 8 + 8 + 32 + 384, "packed layout expected");

}  // namespace

struct sentinel_verifier {
  sentinel_config cfg;
  size_t N = 0, Ns = 0;
  int cap0 = 0, cap1 = 0;
  int R = 1, units0 = 1, units1 = 1; // workers; entries one iteration can append per level
  int G = 1;                        // streaming CTAs; launches use G + 1
  size_t refresh_smem = 0;          // dynamic shared memory of a launch that may refresh thresholds
  int n_metrics = 3;                // metrics in use; 4 once directions are set
  bool started = false;             // a step was taken or a state imported: the metric set is fixed
  int sw_L = 0;                     // number of directions
  uint16_t *sw_u = nullptr;         // directions, bf16 [sw_L][d]
  float *sw_scratch = nullptr;      // projections and sorted lists
  float *sw_out = nullptr;          // [1+B] distances of the submission being checked
  double *sw_pm[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // per kind: projections of the reference, [B*T][L], current and spare
  bool sw_pm_valid[2] = {false, false};   // they match the reference (not so right after a state import)
  void *ema[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // fp32, or bf16 if bf16
  bool bf16 = false;                // the reference is stored as bf16
  bool shared_ref = false;          // one [T,d] reference for all B samples
  bool chan_ref = false;            // the reference is reduced over the tokens: one [d] vector, or
  bool chan_per_sample = false;     //   one per sample ([B,d])
  float *col_part = nullptr;        // chan_ref: column sums of x per streaming CTA and slot
  size_t ema_elems = 0;             // elements of one reference buffer: B*T*d, T*d if shared_ref, d if chan_ref
  size_t ema_bytes = 0;             // bytes of one reference buffer
  HandleState *hs = nullptr;
  double *hist[2] = {nullptr, nullptr};      // rings, device layout (ring_offset)
  double *sorted[2] = {nullptr, nullptr};    // ascending copies of the windows (sorted_offset)
  unsigned long long *partials = nullptr;
  float *stats[2] = {nullptr, nullptr};
  float *token_buf = nullptr;
  float *token_part = nullptr;      // per-tile token sums, allocated when a row spans several tiles
  void *stage_x = nullptr;          // staging for sentinel_verify_host, allocated on first use
  float *stage_scores = nullptr;
  unsigned *stage_flags = nullptr;
  std::string err;
};

namespace {

int fail(sentinel_verifier *h, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->err = buf; else g_error = buf;
  return code;
}

#define SENTINEL_CUDA(h, call)                                                              \
  do {                                                                                      \
    cudaError_t e_ = (call);                                                                \
    if (e_ != cudaSuccess)                                                                  \
      return fail((h), SENTINEL_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
  } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// doubles of history in a checkpoint blob (and of the ascending copies on the device)
size_t hist_doubles(const sentinel_verifier *h) {
  return (size_t)kNumMetrics * ((size_t)h->cap0 + (size_t)h->cap1);
}

// doubles of the rings on the device: each ring has one step's worth of slots more than its window
size_t ring_doubles(const sentinel_verifier *h) {
  return (size_t)kNumMetrics * ((size_t)ring_size(h->cap0, h->units0) + (size_t)ring_size(h->cap1, h->units1));
}

size_t kind_blob_bytes(const sentinel_verifier *h) {
  return sizeof(BlobKindHead) + hist_doubles(h) * sizeof(double) + h->ema_elems * sizeof(float);
}

Alg5Params alg5_of(const sentinel_config &c, int kind) {
  Alg5Params p;
  p.alpha = c.alpha[kind];
  p.gamma_g = c.gamma_grow[kind];
  p.gamma_s = c.gamma_shrink[kind];
  p.lambda = c.lambda_min[kind];
  p.eps = c.iqr_eps[kind];
  p.shrink_ratio = c.shrink_ratio;
  p.n_max = c.n_max[kind];
  p.pad = 0;
  return p;
}

// How many CTAs stream: every resident slot but the one of CTA 0, never more than there are
// rows.  A CTA's rows may straddle one sample boundary at most, which needs G >= B.  `occ` is the
// number of CTAs of the kernel(s) to be launched that an SM keeps resident, as resident_ctas()
// found it for their CTA size and shared memory.
int streaming_ctas(int device, int occ, int B, int T, std::string *err) {
  int sms = 0;
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (e != cudaSuccess || sms < 1 || occ < 1) {
    if (err) *err = std::string("occupancy query failed: ") + cudaGetErrorString(e);
    return -1;
  }
  long long G = (long long)sms * occ - 1;
  const long long rows = (long long)B * T;
  if (G > rows) G = rows;
  if (G < B) {
    if (err) *err = "this device keeps fewer CTAs resident than the tensor has samples";
    return -1;
  }
  return (int)G;
}

// Resident CTAs per SM of one kernel as it will be launched (its CTA size, its dynamic shared
// memory); -1 on failure.  `lowest` carries the minimum over several kernels.
template <typename K>
void resident_ctas(K kernel, int threads, size_t smem, int *lowest, cudaError_t *status) {
  int occ = 0;
  if (*status == cudaSuccess && smem > 48u * 1024u)
    *status = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (*status == cudaSuccess) *status = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, threads, smem);
  if (*status == cudaSuccess && (*lowest < 0 || occ < *lowest)) *lowest = occ;
}

// the stateless distance: stream_kernel_t<false, false> with no dynamic shared memory
int distance_ctas(int device, int B, int T, std::string *err) {
  int occ = -1;
  cudaError_t e = cudaSuccess;
  resident_ctas(stream_kernel_t<false, false>, kThreads, 0, &occ, &e);
  if (e != cudaSuccess) {
    if (err) *err = std::string("occupancy query failed: ") + cudaGetErrorString(e);
    return -1;
  }
  return streaming_ctas(device, occ, B, T, err);
}

// The stateless entry points take their scratch from the device's default memory pool.  By
// default that pool hands everything back to the driver whenever the stream is synchronised, so
// the next call pays for a fresh driver allocation; keeping a little memory cached avoids that.
// Only ever raises the threshold, once per device.
void keep_pool_warm(int device) {
  static std::mutex mu;
  static bool done[64] = {false};
  std::lock_guard<std::mutex> lock(mu);
  if (device < 0 || device >= 64 || done[device]) return;
  done[device] = true;
  cudaMemPool_t pool;
  if (cudaDeviceGetDefaultMemPool(&pool, device) != cudaSuccess) { cudaGetLastError(); return; }
  unsigned long long cur = 0, want = 64ull << 20;
  if (cudaMemPoolGetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &cur) == cudaSuccess && cur < want)
    cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &want);
  cudaGetLastError();
}

int tiles_per_row(int d) { return (((d + 7) >> 3) + 32 * kUnroll - 1) / (32 * kUnroll); }

int check_shape(sentinel_verifier *h, int B, int T, int d, bool vector_path = true) {
  if (B < 1 || T < 1 || d < 1) return fail(h, SENTINEL_ERR_INVALID_ARG, "B, T, d must be positive (got %d, %d, %d)", B, T, d);
  if (vector_path && d % 8 != 0) return fail(h, SENTINEL_ERR_UNALIGNED, "d = %d is not a multiple of 8", d);
  if (B > SENTINEL_MAX_B) return fail(h, SENTINEL_ERR_UNSUPPORTED, "B = %d exceeds SENTINEL_MAX_B = %d", B, SENTINEL_MAX_B);
  return SENTINEL_OK;
}

int check_call(sentinel_verifier *h, const void *x, int kind, int B, int T, int d) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!x) return fail(h, SENTINEL_ERR_INVALID_ARG, "x is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "kind %d is neither ACT nor GRAD", kind);
  if (B != h->cfg.B || T != h->cfg.T || d != h->cfg.d)
    return fail(h, SENTINEL_ERR_SHAPE_MISMATCH, "shape [%d,%d,%d] differs from the handle's [%d,%d,%d]", B, T, d, h->cfg.B, h->cfg.T, h->cfg.d);
  if (d % 8 != 0) return fail(h, SENTINEL_ERR_UNALIGNED, "d = %d is not a multiple of 8: use the _strided entry points", d);
  if (!aligned16(x)) return fail(h, SENTINEL_ERR_UNALIGNED, "x is not 16-byte aligned");
  return SENTINEL_OK;
}

// the strided entry points: any d, rows row_stride elements apart, 2-byte alignment
int check_call_strided(sentinel_verifier *h, const void *x, int kind, int B, int T, int d, long long row_stride) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!x) return fail(h, SENTINEL_ERR_INVALID_ARG, "x is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "kind %d is neither ACT nor GRAD", kind);
  if (B != h->cfg.B || T != h->cfg.T || d != h->cfg.d)
    return fail(h, SENTINEL_ERR_SHAPE_MISMATCH, "shape [%d,%d,%d] differs from the handle's [%d,%d,%d]", B, T, d, h->cfg.B, h->cfg.T, h->cfg.d);
  if (row_stride < d) return fail(h, SENTINEL_ERR_INVALID_ARG, "row_stride = %lld is smaller than d = %d", row_stride, d);
  if (reinterpret_cast<uintptr_t>(x) & 1u) return fail(h, SENTINEL_ERR_UNALIGNED, "x is not 2-byte aligned");
  if (h->sw_u) return fail(h, SENTINEL_ERR_UNSUPPORTED, "the sliced Wasserstein metric reads dense rows: a verifier with directions takes no strided tensor");
  if (h->shared_ref || h->chan_ref) return fail(h, SENTINEL_ERR_UNSUPPORTED, "a verifier with a [T,d] or [d] reference takes no strided tensor");
  return SENTINEL_OK;
}

StreamArgs make_args(sentinel_verifier *h, const void *x, int kind, int mode, float *scores, unsigned *flags) {
  StreamArgs a;
  memset(&a, 0, sizeof a);
  a.x = static_cast<const uint16_t *>(x);
  a.ema[0] = h->ema[kind][0];
  a.ema[1] = h->ema[kind][1];
  a.hs = h->hs;
  a.hist = h->hist[kind];
  a.sorted = h->sorted[kind];
  a.partials = h->partials;
  a.ticket = &h->hs->ticket;
  a.scores_out = scores;
  a.flags_out = flags;
  a.stats_out = h->stats[kind];
  a.token_out = h->token_buf;
  a.token_part = h->token_part;
  a.B = h->cfg.B; a.T = h->cfg.T; a.d = h->cfg.d;
  a.G = h->G;
  a.mode = mode;
  a.kind = kind;
  a.beta = (float)h->cfg.beta[kind];
  a.one_minus_beta = (float)(1.0 - h->cfg.beta[kind]);
  a.cap0 = h->cap0; a.cap1 = h->cap1;
  a.units0 = h->units0; a.units1 = h->units1;
  a.R = h->R;
  a.x_row_stride = h->cfg.d;
  a.a5 = alg5_of(h->cfg, kind);
  a.severe_mult = h->cfg.severe_mult;
  a.ban_violations = h->cfg.ban_violations;
  a.forgiveness_steps = h->cfg.forgiveness_steps;
  a.metric_mask = h->cfg.metric_mask;
  a.ema_bf16 = h->bf16 ? 1 : 0;
  a.n_metrics = h->n_metrics;
  a.sw = h->sw_out;                 // nullptr until directions are set
  a.defer_commit = h->chan_ref ? 1 : 0;
  a.ref_per_sample = h->chan_per_sample ? 1 : 0;
  a.col_part = h->col_part;
  // what the checked build compares indices with
  a.x_extent = h->shared_ref ? (long long)h->Ns : (long long)h->N;    // (a [T,d] reference: per sample slice)
  a.ref_extent = (long long)h->ema_elems;
  a.partials_words = (long long)(h->shared_ref ? h->cfg.B : h->R) * h->G * kSegsPerCta * kSlotWords;
  a.ring_doubles = (long long)ring_doubles(h);
  a.sorted_doubles = (long long)hist_doubles(h);
  a.col_floats = h->chan_ref ? (long long)h->G * kSegsPerCta * channel_slots(h->cfg.d) * kStripe : 0;
  return a;
}

int launch(sentinel_verifier *h, const StreamArgs &a, int grid, cudaStream_t s, bool scalar = false) {
  // launched with programmatic stream serialization: the grid may be set up while the previous
  // kernel on the stream drains; every CTA waits for that kernel before it reads anything
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)grid);
  lc.blockDim = dim3(kThreads);
  lc.dynamicSmemBytes = h->refresh_smem;
  lc.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  if (h->chan_ref) {                               // x alone streams; the reference moves in a second launch
    lc.blockDim = dim3(kChanThreads);
    lc.dynamicSmemBytes = std::max(lc.dynamicSmemBytes, channel_smem_bytes());      // the warps' staging rings
    if (h->chan_per_sample) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, channel_ref_kernel<true>, a));
    else SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, channel_ref_kernel<false>, a));
    cudaLaunchConfig_t lm = lc;
    lm.gridDim = dim3((unsigned)((h->cfg.d + kChannelMeanCols - 1) / kChannelMeanCols), h->chan_per_sample ? (unsigned)h->cfg.B : 1u);
    lm.blockDim = dim3(kChannelMeanCols * kChannelMeanGroups);
    lm.dynamicSmemBytes = 0;
    SENTINEL_CUDA(h, cudaLaunchKernelEx(&lm, channel_mean_kernel, h->hs, a.kind, static_cast<float *>(a.ema[0]),
                                        static_cast<float *>(a.ema[1]), static_cast<const float *>(h->col_part), a.x,
                                        h->G, h->cfg.B, h->cfg.T, h->cfg.d, h->chan_per_sample ? 1 : 0, a.beta, a.one_minus_beta));
    return SENTINEL_OK;
  }
  if (h->shared_ref) {                             // the samples in the workers' place (vector rows only)
    ReplicaArgs ra;
    memset(&ra, 0, sizeof ra);
    ra.s = a;
    for (int b = 0; b < h->cfg.B; ++b) ra.xs[b] = a.x + (size_t)b * h->Ns;
    ra.partials = h->partials;
    if (h->cfg.B <= kFewSets) {
      lc.blockDim = dim3(kFewThreads);
      lc.dynamicSmemBytes = std::max(lc.dynamicSmemBytes, few_smem_bytes());   // the threads' fp64 sums
      SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, shared_ref_kernel<true>, ra));
    } else {
      SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, shared_ref_kernel<false>, ra));
    }
    return SENTINEL_OK;
  }
  // strided rows: the funnel-shift variant of the vector path when the width allows it, else scalar
  const bool shifted = scalar && h->cfg.d % 8 == 0;
  if (h->bf16) {
    if (shifted) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<false, true, true>, a));
    else if (scalar) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<true, true>, a));
    else SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<false, true>, a));
  } else {
    if (shifted) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<false, false, true>, a));
    else if (scalar) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<true, false>, a));
    else SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, stream_kernel_t<false, false>, a));
  }
  return SENTINEL_OK;
}

int run_refresh(sentinel_verifier *h, cudaStream_t s) {
  refresh_kernel<<<1, kThreads, h->refresh_smem, s>>>(h->hs, h->hist[0], h->hist[1], h->sorted[0], h->sorted[1],
                                                      h->cap0, h->cap1, h->units0, h->units1, h->n_metrics,
                                                      alg5_of(h->cfg, 0), alg5_of(h->cfg, 1));
  SENTINEL_CUDA(h, cudaGetLastError());
  return SENTINEL_OK;
}

struct DeviceGuard {   // restores the caller's current device
  int prev = -1;
  cudaError_t status;
  explicit DeviceGuard(int dev) {
    status = cudaGetDevice(&prev);
    if (status == cudaSuccess && prev != dev) status = cudaSetDevice(dev);
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// ---------------------------------------------------------------------------------------------
// sliced Wasserstein distance: the chain of launches, shared by the stateless entry point and
// by verifiers that carry it as their fourth metric

// What a verifier adds to the projection launch: its own projections of the reference (kept up
// to date through the linearity of Eq. 1) and the coefficients of that update.
struct ProjectionState {
  double *pm0 = nullptr, *pm1 = nullptr;   // [rows][L] each; nullptr: stateless
  bool incremental = false;                // take P(m) from the buffers instead of reading m
  float beta = 0.f, one_minus_beta = 0.f;
};

// One launch of the chain, with programmatic stream serialization (see chain_entry()).
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(block);
  lc.dynamicSmemBytes = smem;
  lc.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

template <int L, int kT, bool kRefOnly, bool kBf16>
cudaError_t projection_occupancy(size_t smem, int *occ) {
  cudaError_t e = cudaFuncSetAttribute(swd_project_kernel<L, kT, kRefOnly, kBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(occ, swd_project_kernel<L, kT, kRefOnly, kBf16>, kT, smem);
}

template <int L, bool kRefOnly = false, bool kBf16 = false>
cudaError_t launch_projection(const uint16_t *x, const void *m0, const void *m1, const int *active, const int *skip,
                              const uint16_t *u, float *proj, long long rows, int d, int sms, const ProjectionState &ps,
                              cudaStream_t s) {
  const size_t smem = (size_t)L * d * sizeof(uint16_t);
  int occ_small = 0, occ_large = 0;
  cudaError_t e = projection_occupancy<L, 512, kRefOnly, kBf16>(smem, &occ_small);
  if (e != cudaSuccess) return e;
  e = projection_occupancy<L, 768, kRefOnly, kBf16>(smem, &occ_large);
  if (e != cudaSuccess) return e;
  const bool large = occ_large * 768 > occ_small * 512;
  const int threads = large ? 768 : 512, occ = large ? occ_large : occ_small;
  if (occ < 1) return cudaErrorInvalidConfiguration;
  long long grid = (long long)sms * occ;
  const long long need = (rows + threads / 32 - 1) / (threads / 32);
  if (grid > need) grid = need;
  if (large)
    return launch_chained(swd_project_kernel<L, 768, kRefOnly, kBf16>, (unsigned)grid, 768, smem, s, x, m0, m1, active, skip, u, proj,
                          rows, d, ps.pm0, ps.pm1, ps.beta, ps.one_minus_beta);
  return launch_chained(swd_project_kernel<L, 512, kRefOnly, kBf16>, (unsigned)grid, 512, smem, s, x, m0, m1, active, skip, u, proj,
                        rows, d, ps.pm0, ps.pm1, ps.beta, ps.one_minus_beta);
}

// x alone, on the tensor cores: the reference's projections come from the verifier's own buffers
cudaError_t launch_projection_mma(const uint16_t *x, const int *active, const int *skip, const uint16_t *u, float *proj,
                                  long long rows, int d, int L, int sms, const ProjectionState &ps, cudaStream_t s) {
  const size_t smem = (size_t)L * swd_mma_stride(d >> 3) * sizeof(uint4);
  const long long n_tasks = (rows + 15) / 16;
  const unsigned grid = (unsigned)(n_tasks < sms ? n_tasks : sms);
  cudaError_t e;
  if (L == 16) {
    e = cudaFuncSetAttribute(swd_project_mma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 210 * 1024);
    if (e != cudaSuccess) return e;
    return launch_chained(swd_project_mma_kernel<2>, grid, kSwdMmaThreads, smem, s, x, active, skip, u, proj, rows, d, L,
                          ps.pm0, ps.pm1, ps.beta, ps.one_minus_beta);
  } else {
    e = cudaFuncSetAttribute(swd_project_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 210 * 1024);
    if (e != cudaSuccess) return e;
    return launch_chained(swd_project_mma_kernel<1>, grid, kSwdMmaThreads, smem, s, x, active, skip, u, proj, rows, d, L,
                          ps.pm0, ps.pm1, ps.beta, ps.one_minus_beta);
  }
}

// x and the stored reference (or the reference alone) on the tensor cores.  *fits = false, and
// nothing is launched, if the directions and the warps' partial sums do not fit in shared memory
// together (the caller then takes swd_project_kernel).
template <int NB, bool kWithX, bool kBf16>
cudaError_t launch_projection_ref_mma_nb(const uint16_t *x, const void *m0, const void *m1, const int *active, const int *skip,
                                         const uint16_t *u, float *proj, long long rows, int d, int L, int sms,
                                         const ProjectionState &ps, cudaStream_t s, bool *fits) {
  const size_t smem = (size_t)L * swd_mma_stride(d >> 3) * sizeof(uint4) +
                      (size_t)kSwdRefWarps * (kWithX ? 2 : 1) * NB * 4 * 32 * sizeof(float);
  *fits = smem <= 227u * 1024u;
  if (!*fits) return cudaSuccess;
  const long long n_tasks = (rows + 15) / 16;
  const unsigned grid = (unsigned)(n_tasks < sms ? n_tasks : sms);
  cudaError_t e = cudaFuncSetAttribute(swd_project_ref_mma_kernel<NB, kWithX, kBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  return launch_chained(swd_project_ref_mma_kernel<NB, kWithX, kBf16>, grid, kSwdRefThreads, smem, s, x, m0, m1, active, skip, u,
                        proj, rows, d, L, ps.pm0, ps.pm1, ps.beta, ps.one_minus_beta);
}

template <bool kWithX>
cudaError_t launch_projection_ref_mma(const uint16_t *x, const void *m0, const void *m1, bool ref_bf16, const int *active,
                                      const int *skip, const uint16_t *u, float *proj, long long rows, int d, int L, int sms,
                                      const ProjectionState &ps, cudaStream_t s, bool *fits) {
  if (L == 16) {
    if (ref_bf16) return launch_projection_ref_mma_nb<2, kWithX, true>(x, m0, m1, active, skip, u, proj, rows, d, L, sms, ps, s, fits);
    return launch_projection_ref_mma_nb<2, kWithX, false>(x, m0, m1, active, skip, u, proj, rows, d, L, sms, ps, s, fits);
  }
  if (ref_bf16) return launch_projection_ref_mma_nb<1, kWithX, true>(x, m0, m1, active, skip, u, proj, rows, d, L, sms, ps, s, fits);
  return launch_projection_ref_mma_nb<1, kWithX, false>(x, m0, m1, active, skip, u, proj, rows, d, L, sms, ps, s, fits);
}

// floats of scratch: the projections, the sorted lists and one more buffer of that size for the
// merge rounds (2L lists of B*T each; the projections are free again by then and serve as the
// other buffer), then swd_w1_kernel's per-CTA sums (doubles) and its ticket word
size_t swd_scratch_floats(int L, int B, int T) {
  return (size_t)3 * 2 * L * ((size_t)B * T) + 2 * swd_w1_partials(L, B, T) + 4;
}

int check_swd_shape(sentinel_verifier *h, int L, int T, int d) {
  if (L != 4 && L != 8 && L != 16) return fail(h, SENTINEL_ERR_UNSUPPORTED, "L = %d: the number of directions must be 4, 8 or 16", L);
  if ((size_t)L * d * sizeof(uint16_t) > 200u * 1024u) return fail(h, SENTINEL_ERR_UNSUPPORTED, "L*d = %d*%d directions do not fit in 200 KiB of shared memory", L, d);
  if (T > kSwdMaxTokensPerSample) return fail(h, SENTINEL_ERR_UNSUPPORTED, "T = %d exceeds the %d tokens sorted per sample", T, kSwdMaxTokensPerSample);
  return SENTINEL_OK;
}

// out[0] = the whole tensor, out[1+b] = sample b.  The reference is m1 if *active != 0, else m0;
// nothing runs if *skip != 0 (both read on the device; either may be nullptr).
// (ref_bf16: m0 / m1 hold bf16 instead of fp32)
cudaError_t run_swd(const uint16_t *x, const void *m0, const void *m1, bool ref_bf16, const int *active, const int *skip,
                    const uint16_t *u, int L, int B, int T, int d, int sms, float *scratch, float *out,
                    const ProjectionState &ps, cudaStream_t s) {
  const long long rows = (long long)B * T;
  const size_t list_floats = (size_t)2 * L * rows;        // L lists for x, L for m
  float *proj = scratch, *sorted = proj + list_floats, *spare = sorted + list_floats;
  double *partial = reinterpret_cast<double *>(spare + list_floats);      // (list_floats is even: 8-byte aligned)
  unsigned *ticket = reinterpret_cast<unsigned *>(partial + swd_w1_partials(L, B, T));
  cudaError_t e;
  if (ps.incremental) {
    e = launch_projection_mma(x, active, skip, u, proj, rows, d, L, sms, ps, s);
  } else {
    bool fits = false;
    e = launch_projection_ref_mma<true>(x, m0, m1, ref_bf16, active, skip, u, proj, rows, d, L, sms, ps, s, &fits);
    if (e == cudaSuccess && !fits) {
      if (ref_bf16) {
        if (L == 4) e = launch_projection<4, false, true>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
        else if (L == 8) e = launch_projection<8, false, true>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
        else e = launch_projection<16, false, true>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
      } else {
        if (L == 4) e = launch_projection<4>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
        else if (L == 8) e = launch_projection<8>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
        else e = launch_projection<16>(x, m0, m1, active, skip, u, proj, rows, d, sms, ps, s);
      }
    }
  }
  if (e != cudaSuccess) return e;
  // few lists: each sample's list is sorted as two halves on twice as many SMs, and a merge round follows
  const int pieces = (T % 2 == 0 && T >= 1024 && 2 * L * B * 2 <= sms) ? 2 : 1;
  int npad = 8;
  while (npad < T / pieces) npad <<= 1;
  const size_t smem = (size_t)npad * sizeof(float);
  e = cudaFuncSetAttribute(swd_sort_samples_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSwdMaxTokensPerSample * (int)sizeof(float));
  if (e != cudaSuccess) return e;
  SwdExtents ext;                                  // (from the layout of the scratch, not from the kernels' own arithmetic)
  ext.list_floats = (long long)(sorted - proj);
  ext.partial_doubles = (long long)(reinterpret_cast<double *>(ticket) - partial);
  e = launch_chained(swd_sort_samples_kernel, 2u * L * B * pieces, kSwdSortThreads, smem, s, proj, sorted, ticket, B, T, pieces, L,
                     rows, skip, ext);
  if (e != cudaSuccess) return e;
  const long long span_tasks = (rows + kSwdMergeSpan - 1) / kSwdMergeSpan * 2 * L;
  const unsigned merge_grid = (unsigned)((span_tasks + kSwdW1Threads - 1) / kSwdW1Threads);
  // the three buffers: `samples` holds the samples' sorted lists until swd_w1_kernel has read them,
  // the merge rounds (all but the last, which swd_w1_kernel does itself) alternate between the other two
  const float *samples = sorted;
  float *free_a = spare, *free_b = proj;
  if (pieces == 2) {
    e = launch_chained(swd_merge_kernel, merge_grid, kSwdW1Threads, 0, s, sorted, spare, rows, (long long)(T / 2), 2 * L, skip, ext);
    if (e != cudaSuccess) return e;
    samples = spare;
    free_a = proj;
    free_b = sorted;
  }
  const float *runs = samples;
  long long run_len = T;
  while (2 * run_len < rows) {
    e = launch_chained(swd_merge_kernel, merge_grid, kSwdW1Threads, 0, s, runs, free_a, rows, run_len, 2 * L, skip, ext);
    if (e != cudaSuccess) return e;
    runs = free_a;
    float *t = free_a; free_a = free_b; free_b = t;
    run_len *= 2;
  }
  const unsigned grid = (unsigned)((B > 1 ? L * swd_w1_chunks(rows) : 0) + L * B * swd_w1_chunks(T));
  return launch_chained(swd_w1_kernel, grid, kSwdW1Threads, 0, s, samples, runs, run_len, partial, ticket, out, B, T, L, rows, skip, ext);
}

// A verifier with directions: the distances of this submission against the reference in force,
// left in h->sw_out for the streaming launch that follows on the same stream.
int run_handle_swd(sentinel_verifier *h, const void *x, int kind, int worker, bool may_skip, cudaStream_t s) {
  if (!h->sw_u) return SENTINEL_OK;
  int sms = 0;
  SENTINEL_CUDA(h, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->cfg.device));
  ProjectionState ps;
  ps.pm0 = h->sw_pm[kind][0];
  ps.pm1 = h->sw_pm[kind][1];
  ps.beta = (float)h->cfg.beta[kind];
  ps.one_minus_beta = (float)(1.0 - h->cfg.beta[kind]);
  // One submission per update: the reference's projections follow it (Eq. 1 is linear).  Several
  // workers: run_reference_projection has just put P(m) into the current buffer; what the x-only
  // launch writes into the spare one is never adopted.
  ps.incremental = h->R == 1 ? h->sw_pm_valid[kind] : true;
  // A bf16 reference is rounded when it is stored, so its projections do not follow the recursion:
  // a single-submission verifier projects it afresh every step (2 + 2 B/element read instead of 2).
  if (h->bf16 && h->R == 1) { ps.incremental = false; ps.pm0 = ps.pm1 = nullptr; }
  SENTINEL_CUDA(h, run_swd(static_cast<const uint16_t *>(x), h->ema[kind][0], h->ema[kind][1], h->bf16,
                           &h->hs->kind[kind].active,
                           may_skip ? &h->hs->banned[worker] : nullptr, h->sw_u, h->sw_L, h->cfg.B, h->cfg.T,
                           h->cfg.d, sms, h->sw_scratch, h->sw_out + (size_t)worker * (1 + h->cfg.B), ps, s));
  if (h->R == 1 && !h->bf16) h->sw_pm_valid[kind] = true;      // that launch (re)computed them from m if they were stale
  return SENTINEL_OK;
}

// A verifier with directions that follows several workers: the reference's projections, once per
// iteration, for all workers' chains to read.
int run_reference_projection(sentinel_verifier *h, int kind, cudaStream_t s) {
  if (!h->sw_u || h->R == 1) return SENTINEL_OK;
  int sms = 0;
  SENTINEL_CUDA(h, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->cfg.device));
  ProjectionState ps;
  ps.pm0 = h->sw_pm[kind][0];
  ps.pm1 = h->sw_pm[kind][1];
  const void *m0 = h->ema[kind][0], *m1 = h->ema[kind][1];
  const int *active = &h->hs->kind[kind].active;
  const long long rows = (long long)h->cfg.B * h->cfg.T;
  bool fits = false;
  cudaError_t e = launch_projection_ref_mma<false>(nullptr, m0, m1, h->bf16, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d,
                                                   h->sw_L, sms, ps, s, &fits);
  if (e == cudaSuccess && !fits) {
    if (h->bf16) {
      if (h->sw_L == 4) e = launch_projection<4, true, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
      else if (h->sw_L == 8) e = launch_projection<8, true, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
      else e = launch_projection<16, true, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
    } else if (h->sw_L == 4) e = launch_projection<4, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
    else if (h->sw_L == 8) e = launch_projection<8, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
    else e = launch_projection<16, true>(nullptr, m0, m1, active, nullptr, h->sw_u, nullptr, rows, h->cfg.d, sms, ps, s);
  }
  SENTINEL_CUDA(h, e);
  return SENTINEL_OK;
}

// a single submission (worker slot 0), whatever the number of workers the handle follows
int run_single_swd(sentinel_verifier *h, const void *x, int kind, cudaStream_t s) {
  int rc = run_reference_projection(h, kind, s);
  if (rc) return rc;
  return run_handle_swd(h, x, kind, 0, false, s);
}

void free_all(sentinel_verifier *h) {
  for (int k = 0; k < 2; ++k) {
    for (int j = 0; j < 2; ++j) cudaFree(h->ema[k][j]);
    cudaFree(h->hist[k]);
    cudaFree(h->sorted[k]);
    cudaFree(h->stats[k]);
  }
  cudaFree(h->hs);
  cudaFree(h->partials);
  cudaFree(h->token_part);
  cudaFree(h->col_part);
  cudaFree(h->stage_x);
  cudaFree(h->stage_scores);
  cudaFree(h->stage_flags);
  cudaFree(h->sw_u);
  cudaFree(h->sw_scratch);
  cudaFree(h->sw_out);
  for (int k = 0; k < 2; ++k)
    for (int j = 0; j < 2; ++j) cudaFree(h->sw_pm[k][j]);
}

}  // namespace

extern "C" {

int sentinel_default_config(sentinel_config *cfg) {
  if (!cfg) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "cfg is NULL");
  memset(cfg, 0, sizeof *cfg);
  cfg->beta[0] = 0.90;         cfg->beta[1] = 0.80;
  cfg->k0[0] = 1.5;            cfg->k0[1] = 3.0;
  cfg->alpha[0] = 1e-4;        cfg->alpha[1] = 1e-3;
  cfg->n_max[0] = 10;          cfg->n_max[1] = 10;
  cfg->gamma_grow[0] = 1.1;    cfg->gamma_grow[1] = 1.01;
  cfg->gamma_shrink[0] = 0.9;  cfg->gamma_shrink[1] = 0.99;
  cfg->lambda_min[0] = 0.15;   cfg->lambda_min[1] = 0.05;
  cfg->iqr_eps[0] = 1e-3;      cfg->iqr_eps[1] = 5e-5;
  cfg->shrink_ratio = 0.5;
  cfg->severe_mult = 100.0;
  cfg->window_steps = 100;
  cfg->ban_violations = 5;
  cfg->forgiveness_steps = 100;
  cfg->metric_mask = 15u;
  cfg->n_workers = 1;
  return SENTINEL_OK;
}

int sentinel_verifier_create(const sentinel_config *cfg, sentinel_verifier **out) {
  if (!cfg || !out) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "cfg or out is NULL");
  *out = nullptr;
  int rc = check_shape(nullptr, cfg->B, cfg->T, cfg->d, false);   // d % 8 != 0: strided entry points only
  if (rc) return rc;
  for (int k = 0; k < 2; ++k) {
    if (!(cfg->beta[k] >= 0.0 && cfg->beta[k] < 1.0)) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "beta[%d] = %g is outside [0,1)", k, cfg->beta[k]);
    if (!(cfg->k0[k] > 0.0) || !(cfg->gamma_grow[k] > 1.0) || !(cfg->gamma_shrink[k] > 0.0 && cfg->gamma_shrink[k] < 1.0) ||
        !(cfg->alpha[k] >= 0.0) || cfg->n_max[k] < 0 || !(cfg->lambda_min[k] >= 0.0) || !(cfg->iqr_eps[k] >= 0.0))
      return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "threshold parameters of kind %d are out of range", k);
  }
  if (cfg->window_steps < 1 || cfg->ban_violations < 1 || cfg->forgiveness_steps < 1 || !(cfg->severe_mult > 0.0) || !(cfg->shrink_ratio >= 0.0))
    return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "window_steps, ban_violations, forgiveness_steps, severe_mult must be positive");
  if (cfg->n_workers < 1 || cfg->n_workers > SENTINEL_MAX_WORKERS)
    return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "n_workers = %d is outside 1..%d", cfg->n_workers, SENTINEL_MAX_WORKERS);
  if (cfg->ema_bf16 != 0 && cfg->ema_bf16 != 1) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "ema_bf16 must be 0 or 1, got %d", cfg->ema_bf16);
  if (cfg->ref_over_batch != 0 && cfg->ref_over_batch != 1) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "ref_over_batch must be 0 or 1, got %d", cfg->ref_over_batch);
  if (cfg->ref_over_batch && (cfg->n_workers != 1 || cfg->ema_bf16 || (cfg->B > kMaxWorkers && !cfg->ref_over_tokens) || cfg->d % 8 != 0))
    return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "a [T,d] reference needs n_workers = 1, an fp32 reference, B <= %d and d a multiple of 8", kMaxWorkers);
  if (cfg->ref_over_tokens != 0 && cfg->ref_over_tokens != 1) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "ref_over_tokens must be 0 or 1, got %d", cfg->ref_over_tokens);
  if (cfg->ref_over_tokens && (cfg->n_workers != 1 || cfg->ema_bf16 || cfg->d % 8 != 0))
    return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "a reference reduced over the tokens needs n_workers = 1, an fp32 reference and d a multiple of 8");
  if ((long long)cfg->window_steps * cfg->n_workers * (cfg->B + 1) > SENTINEL_MAX_WINDOW)
    return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "window_steps*n_workers*(B+1) = %lld exceeds SENTINEL_MAX_WINDOW = %d",
                (long long)cfg->window_steps * cfg->n_workers * (cfg->B + 1), SENTINEL_MAX_WINDOW);
  int ndev = 0;
  SENTINEL_CUDA(nullptr, cudaGetDeviceCount(&ndev));
  if (cfg->device < 0 || cfg->device >= ndev) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "device %d does not exist (%d devices)", cfg->device, ndev);

  DeviceGuard guard(cfg->device);
  SENTINEL_CUDA(nullptr, guard.status);

  sentinel_verifier *h = new (std::nothrow) sentinel_verifier();
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "out of host memory");
  h->cfg = *cfg;
  h->Ns = (size_t)cfg->T * cfg->d;
  h->N = h->Ns * cfg->B;
  h->R = cfg->n_workers;
  h->bf16 = cfg->ema_bf16 != 0;
  h->chan_ref = cfg->ref_over_tokens != 0;
  h->shared_ref = cfg->ref_over_batch != 0 && !h->chan_ref;
  h->chan_per_sample = h->chan_ref && cfg->ref_over_batch == 0;
  h->ema_elems = h->chan_ref ? (size_t)cfg->d * (h->chan_per_sample ? (size_t)cfg->B : 1u) : h->shared_ref ? h->Ns : h->N;
  h->ema_bytes = h->ema_elems * (h->bf16 ? sizeof(uint16_t) : sizeof(float));
  h->units0 = h->R;                       // the window spans window_steps iterations of all workers
  h->units1 = h->R * cfg->B;
  h->cap0 = cfg->window_steps * h->units0;
  h->cap1 = cfg->window_steps * h->units1;
  h->refresh_smem = refresh_smem_doubles(h->cap0, h->cap1, h->units0, h->units1, h->n_metrics) * sizeof(double);
  if (h->refresh_smem > 200u * 1024u) {
    const size_t need = h->refresh_smem;
    delete h;
    return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "the windows' working copies need %zu bytes of shared memory, 204800 are available", need);
  }
  {   // the windows' working copies may exceed the 48 KiB a kernel gets without asking
    const int most = 200 * 1024;
    cudaError_t ae = cudaFuncSetAttribute(stream_kernel_t<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(stream_kernel_t<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(stream_kernel_t<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(stream_kernel_t<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(stream_kernel_t<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(stream_kernel_t<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(refresh_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(replica_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(replica_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(replica_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(replica_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(shared_ref_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(shared_ref_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(channel_ref_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae == cudaSuccess) ae = cudaFuncSetAttribute(channel_ref_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    if (ae != cudaSuccess) { delete h; return fail(nullptr, SENTINEL_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(ae)); }
  }
  std::string oerr;
  {
    // Every kernel this handle can launch, with the CTA size and the most dynamic shared memory it
    // can be launched with (the windows' working copies for four metrics, if directions may still
    // be set): G follows the one that keeps the fewest CTAs resident.
    size_t smem = h->refresh_smem;
    const size_t smem4 = refresh_smem_doubles(h->cap0, h->cap1, h->units0, h->units1, kNumMetrics) * sizeof(double);
    if (smem4 <= 200u * 1024u) smem = smem4;
    int occ = -1;
    cudaError_t oe = cudaSuccess;
    if (h->chan_ref) {
      const size_t sm = std::max(smem, channel_smem_bytes());
      if (h->chan_per_sample) resident_ctas(channel_ref_kernel<true>, kChanThreads, sm, &occ, &oe);
      else resident_ctas(channel_ref_kernel<false>, kChanThreads, sm, &occ, &oe);
    } else if (h->shared_ref) {
      if (cfg->B <= kFewSets) resident_ctas(shared_ref_kernel<true>, kFewThreads, std::max(smem, few_smem_bytes()), &occ, &oe);
      else resident_ctas(shared_ref_kernel<false>, kThreads, smem, &occ, &oe);
    } else {
      if (h->R > 1 && h->R <= kFewSets && h->bf16) resident_ctas(replica_kernel<true, true>, kFewThreads, std::max(smem, few_smem_bytes()), &occ, &oe);
      else if (h->R > 1 && h->R <= kFewSets) resident_ctas(replica_kernel<true, false>, kFewThreads, std::max(smem, few_smem_bytes()), &occ, &oe);
      else if (h->R > 1 && h->bf16) resident_ctas(replica_kernel<false, true>, kThreads, smem, &occ, &oe);
      else if (h->R > 1) resident_ctas(replica_kernel<false, false>, kThreads, smem, &occ, &oe);
      if (h->bf16) {
        resident_ctas(stream_kernel_t<false, true>, kThreads, smem, &occ, &oe);
        resident_ctas(stream_kernel_t<true, true>, kThreads, smem, &occ, &oe);
        resident_ctas(stream_kernel_t<false, true, true>, kThreads, smem, &occ, &oe);
      } else {
        resident_ctas(stream_kernel_t<false, false>, kThreads, smem, &occ, &oe);
        resident_ctas(stream_kernel_t<true, false>, kThreads, smem, &occ, &oe);
        resident_ctas(stream_kernel_t<false, false, true>, kThreads, smem, &occ, &oe);
      }
    }
    if (oe != cudaSuccess) { delete h; return fail(nullptr, SENTINEL_ERR_CUDA, "occupancy query failed: %s", cudaGetErrorString(oe)); }
    // (with a [T,d] reference the CTAs share out the T token rows, each with every sample's slice)
    h->G = h->shared_ref ? streaming_ctas(cfg->device, occ, 1, cfg->T, &oerr) : streaming_ctas(cfg->device, occ, cfg->B, cfg->T, &oerr);
  }
  if (h->G < 1) { delete h; return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "%s", oerr.c_str()); }

  cudaError_t e = cudaSuccess;
  auto alloc = [&](void **p, size_t bytes) {
    if (e == cudaSuccess) e = cudaMalloc(p, bytes);
    if (e == cudaSuccess) e = cudaMemset(*p, 0, bytes);
  };
  for (int k = 0; k < 2; ++k) {
    for (int j = 0; j < 2; ++j) alloc(&h->ema[k][j], h->ema_bytes);   // m_0 = 0 (all-zero bits in either format)
    alloc((void **)&h->hist[k], ring_doubles(h) * sizeof(double));
    alloc((void **)&h->sorted[k], hist_doubles(h) * sizeof(double));
    alloc((void **)&h->stats[k], (size_t)(1 + cfg->B) * kNumStats * sizeof(float));
  }
  alloc((void **)&h->partials, (size_t)(h->shared_ref ? cfg->B : h->R) * h->G * kSegsPerCta * kSlotWords * sizeof(unsigned long long));   // per worker / per sample
  if (h->chan_ref) alloc((void **)&h->col_part, (size_t)h->G * kSegsPerCta * channel_slots(cfg->d) * kStripe * sizeof(float));
  alloc((void **)&h->hs, sizeof(HandleState));
  if (e == cudaSuccess) {
    HandleState init;
    memset(&init, 0, sizeof init);
    for (int k = 0; k < 2; ++k)
      for (int L = 0; L < 2; ++L)
        for (int i = 0; i < kNumMetrics; ++i) init.kind[k].thr[L][i][3] = cfg->k0[k];
    e = cudaMemcpy(h->hs, &init, sizeof init, cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    free_all(h);
    delete h;
    return fail(nullptr, SENTINEL_ERR_CUDA, "allocating verifier state failed: %s", cudaGetErrorString(e));
  }
  *out = h;
  return SENTINEL_OK;
}

int sentinel_verify(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T, int d,
                    void *cuda_stream, float *dev_scores_out, unsigned *dev_flags_out) {
  int rc = check_call(h, dev_x, kind, B, T, d);
  if (rc) return rc;
  if (!dev_scores_out || !dev_flags_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "scores_out or flags_out is NULL");
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  h->started = true;
  rc = run_single_swd(h, dev_x, kind, static_cast<cudaStream_t>(cuda_stream));
  if (rc) return rc;
  return launch(h, make_args(h, dev_x, kind, kModeVerify, dev_scores_out, dev_flags_out), h->G + 1,
                static_cast<cudaStream_t>(cuda_stream));
}

int sentinel_update_reference(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T,
                              int d, void *cuda_stream, float *dev_scores_out) {
  int rc = check_call(h, dev_x, kind, B, T, d);
  if (rc) return rc;
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  h->started = true;
  rc = run_single_swd(h, dev_x, kind, static_cast<cudaStream_t>(cuda_stream));
  if (rc) return rc;
  return launch(h, make_args(h, dev_x, kind, kModeWarmup, dev_scores_out, nullptr), h->G + 1,
                static_cast<cudaStream_t>(cuda_stream));
}

int sentinel_verify_strided(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T, int d,
                            long long row_stride, void *cuda_stream, float *dev_scores_out, unsigned *dev_flags_out) {
  int rc = check_call_strided(h, dev_x, kind, B, T, d, row_stride);
  if (rc) return rc;
  if (!dev_scores_out || !dev_flags_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "scores_out or flags_out is NULL");
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  h->started = true;
  StreamArgs a = make_args(h, dev_x, kind, kModeVerify, dev_scores_out, dev_flags_out);
  a.x_row_stride = row_stride;
  a.x_extent = ((long long)B * T - 1) * row_stride + d;
  return launch(h, a, h->G + 1, static_cast<cudaStream_t>(cuda_stream), true);
}

int sentinel_update_reference_strided(sentinel_verifier *h, const void *dev_x, sentinel_kind kind, int B, int T,
                                      int d, long long row_stride, void *cuda_stream, float *dev_scores_out) {
  int rc = check_call_strided(h, dev_x, kind, B, T, d, row_stride);
  if (rc) return rc;
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  h->started = true;
  StreamArgs a = make_args(h, dev_x, kind, kModeWarmup, dev_scores_out, nullptr);
  a.x_row_stride = row_stride;
  a.x_extent = ((long long)B * T - 1) * row_stride + d;
  return launch(h, a, h->G + 1, static_cast<cudaStream_t>(cuda_stream), true);
}

int sentinel_verify_host(sentinel_verifier *h, const void *host_x, sentinel_kind kind, int B, int T,
                         int d, void *cuda_stream, float *host_scores_out, unsigned *host_flags_out) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_x || !host_scores_out || !host_flags_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "a host pointer is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "kind %d is neither ACT nor GRAD", (int)kind);
  if (B != h->cfg.B || T != h->cfg.T || d != h->cfg.d)
    return fail(h, SENTINEL_ERR_SHAPE_MISMATCH, "shape [%d,%d,%d] differs from the handle's [%d,%d,%d]", B, T, d, h->cfg.B, h->cfg.T, h->cfg.d);
  if (d % 8 != 0) return fail(h, SENTINEL_ERR_UNALIGNED, "d = %d is not a multiple of 8: use the _strided entry points", d);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t rows = 1 + (size_t)B;
  if (!h->stage_x) {
    SENTINEL_CUDA(h, cudaMalloc(&h->stage_x, h->N * sizeof(uint16_t)));
    SENTINEL_CUDA(h, cudaMalloc((void **)&h->stage_scores, rows * kNumMetrics * sizeof(float)));
    SENTINEL_CUDA(h, cudaMalloc((void **)&h->stage_flags, rows * sizeof(unsigned)));
  }
  SENTINEL_CUDA(h, cudaMemcpyAsync(h->stage_x, host_x, h->N * sizeof(uint16_t), cudaMemcpyHostToDevice, s));
  h->started = true;
  int rc = run_single_swd(h, h->stage_x, kind, s);
  if (rc) return rc;
  rc = launch(h, make_args(h, h->stage_x, kind, kModeVerify, h->stage_scores, h->stage_flags), h->G + 1, s);
  if (rc) return rc;
  SENTINEL_CUDA(h, cudaMemcpyAsync(host_scores_out, h->stage_scores, rows * h->n_metrics * sizeof(float), cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaMemcpyAsync(host_flags_out, h->stage_flags, rows * sizeof(unsigned), cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));
  return SENTINEL_OK;
}

int sentinel_distance(const void *dev_x, const float *dev_m, int B, int T, int d, int device,
                      void *cuda_stream, float *dev_scores_out, float *dev_stats_out) {
  if (!dev_x || !dev_m || !dev_scores_out) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "x, m or scores_out is NULL");
  int rc = check_shape(nullptr, B, T, d);
  if (rc) return rc;
  if (!aligned16(dev_x) || !aligned16(dev_m)) return fail(nullptr, SENTINEL_ERR_UNALIGNED, "x or m is not 16-byte aligned");
  int ndev = 0;
  SENTINEL_CUDA(nullptr, cudaGetDeviceCount(&ndev));
  if (device < 0 || device >= ndev) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "device %d does not exist", device);
  DeviceGuard guard(device);
  SENTINEL_CUDA(nullptr, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

  std::string oerr;
  const int G = distance_ctas(device, B, T, &oerr);
  if (G < 1) return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "%s", oerr.c_str());
  // scratch: two partial slots per streaming CTA, then the ticket word
  const size_t slot_bytes = (size_t)G * kSegsPerCta * kSlotWords * sizeof(unsigned long long);
  unsigned char *scratch = nullptr;
  keep_pool_warm(device);
  SENTINEL_CUDA(nullptr, cudaMallocAsync((void **)&scratch, slot_bytes + 256, s));
  {
    const cudaError_t me = cudaMemsetAsync(scratch + slot_bytes, 0, 256, s);
    if (me != cudaSuccess) {
      cudaFreeAsync(scratch, s);                       // nothing was launched on it
      return fail(nullptr, SENTINEL_ERR_CUDA, "clearing the scratch failed: %s", cudaGetErrorString(me));
    }
  }

  StreamArgs a;
  memset(&a, 0, sizeof a);
  a.x = static_cast<const uint16_t *>(dev_x);
  a.m_ext = dev_m;
  a.partials = reinterpret_cast<unsigned long long *>(scratch);
  a.ticket = reinterpret_cast<unsigned *>(scratch + slot_bytes);
  a.scores_out = dev_scores_out;
  a.stats_out = dev_stats_out;
  a.B = B; a.T = T; a.d = d; a.G = G;
  a.x_row_stride = d;
  a.x_extent = a.ref_extent = (long long)B * T * d;
  a.partials_words = (long long)G * kSegsPerCta * kSlotWords;
  a.n_metrics = 3;
  a.mode = kModeDistance;
  stream_kernel_t<false, false><<<G + 1, kThreads, 0, s>>>(a);
  cudaError_t le = cudaGetLastError();
  cudaError_t fe = cudaFreeAsync(scratch, s);
  SENTINEL_CUDA(nullptr, le);
  SENTINEL_CUDA(nullptr, fe);
  return SENTINEL_OK;
}

}  // extern "C"

namespace {

int step_replicas(sentinel_verifier *h, const void *const *xs, int kind, unsigned tainted_in, int B, int T, int d,
                  void *cuda_stream, float *scores, unsigned *flags, bool warmup) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!xs) return fail(h, SENTINEL_ERR_INVALID_ARG, "the array of tensors is NULL");
  if (warmup) tainted_in = 0;                        // the warm-up phase has honest workers only
  if (h->R < 32 && (tainted_in >> h->R) != 0) return fail(h, SENTINEL_ERR_INVALID_ARG, "tainted_in names workers beyond n_workers = %d", h->R);
  for (int r = 0; r < h->R; ++r) {
    if ((tainted_in >> r) & 1u) continue;            // not collected: its pointer is not looked at
    int rc = check_call(h, xs[r], kind, B, T, d);
    if (rc) return rc;
  }
  if (!scores || (!warmup && !flags)) return fail(h, SENTINEL_ERR_INVALID_ARG, "scores_out or flags_out is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "kind %d is neither ACT nor GRAD", kind);
  if (B != h->cfg.B || T != h->cfg.T || d != h->cfg.d)
    return fail(h, SENTINEL_ERR_SHAPE_MISMATCH, "shape [%d,%d,%d] differs from the handle's [%d,%d,%d]", B, T, d, h->cfg.B, h->cfg.T, h->cfg.d);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t rows = 1 + (size_t)B;
  h->started = true;
  if (warmup && flags) SENTINEL_CUDA(h, cudaMemsetAsync(flags, 0, h->R * rows * sizeof(unsigned), s));

  ReplicaArgs ra;
  memset(&ra, 0, sizeof ra);
  ra.s = make_args(h, nullptr, kind, warmup ? kModeReplicaWarmup : kModeReplicaVerify, nullptr, nullptr);
  ra.s.sw = nullptr;
  ra.partials = h->partials;
  ra.scores_all = scores;
  ra.flags_all = warmup ? nullptr : flags;
  ra.sw_all = h->sw_out;
  ra.tainted_in = tainted_in;
  WorkerPointers wp;
  memset(&wp, 0, sizeof wp);
  {
    int rc = run_reference_projection(h, kind, s);
    if (rc) return rc;
  }
  for (int r = 0; r < h->R; ++r) {
    if ((tainted_in >> r) & 1u) continue;
    ra.xs[r] = wp.x[r] = static_cast<const uint16_t *>(xs[r]);
    // with directions: every collected worker's distances first, each into its own row block
    int rc = run_handle_swd(h, xs[r], kind, r, !warmup, s);
    if (rc) return rc;
  }
  {   // every worker against the same m_{t-1}, in one launch
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(h->G + 1));
    const bool few = h->R <= kFewSets;              // every worker's sums in registers
    lc.blockDim = dim3(few ? kFewThreads : kThreads);
    lc.dynamicSmemBytes = few ? std::max(h->refresh_smem, few_smem_bytes()) : h->refresh_smem;
    lc.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = 1;
    if (few && h->bf16) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, replica_kernel<true, true>, ra));
    else if (few) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, replica_kernel<true, false>, ra));
    else if (h->bf16) SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, replica_kernel<false, true>, ra));
    else SENTINEL_CUDA(h, cudaLaunchKernelEx(&lc, replica_kernel<false, false>, ra));
  }
  int sms = 0;
  SENTINEL_CUDA(h, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->cfg.device));
  const long long n_chunks = (long long)(h->N / 8);
  long long grid = (long long)sms * 8;
  const long long need = (n_chunks + kReplaceThreads - 1) / kReplaceThreads;
  if (grid > need) grid = need;
  if (h->bf16)
    ema_mean_kernel<true><<<(unsigned)grid, kReplaceThreads, 0, s>>>(
        h->hs, kind, wp, h->ema[kind][0], h->ema[kind][1], n_chunks, h->R, (int)rows, (float)h->cfg.beta[kind],
        (float)(1.0 - h->cfg.beta[kind]), warmup ? 1 : 0, flags);
  else
    ema_mean_kernel<false><<<(unsigned)grid, kReplaceThreads, 0, s>>>(
        h->hs, kind, wp, h->ema[kind][0], h->ema[kind][1], n_chunks, h->R, (int)rows, (float)h->cfg.beta[kind],
        (float)(1.0 - h->cfg.beta[kind]), warmup ? 1 : 0, flags);
  SENTINEL_CUDA(h, cudaGetLastError());
  return SENTINEL_OK;
}

}  // namespace

extern "C" {

int sentinel_verify_replicas(sentinel_verifier *h, const void *const *host_dev_xs, sentinel_kind kind, int B,
                             int T, int d, void *cuda_stream, float *dev_scores_out, unsigned *dev_flags_out) {
  return step_replicas(h, host_dev_xs, kind, 0u, B, T, d, cuda_stream, dev_scores_out, dev_flags_out, false);
}

int sentinel_verify_replicas_tainted(sentinel_verifier *h, const void *const *host_dev_xs, sentinel_kind kind,
                                     unsigned tainted_in, int B, int T, int d, void *cuda_stream,
                                     float *dev_scores_out, unsigned *dev_flags_out) {
  return step_replicas(h, host_dev_xs, kind, tainted_in, B, T, d, cuda_stream, dev_scores_out, dev_flags_out, false);
}

int sentinel_skip_tainted(sentinel_verifier *h, sentinel_kind kind, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "kind %d is neither ACT nor GRAD", (int)kind);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  h->started = true;
  skip_tainted_kernel<<<1, 1, 0, static_cast<cudaStream_t>(cuda_stream)>>>(h->hs, (int)kind);
  SENTINEL_CUDA(h, cudaGetLastError());
  return SENTINEL_OK;
}

int sentinel_update_reference_replicas(sentinel_verifier *h, const void *const *host_dev_xs, sentinel_kind kind,
                                       int B, int T, int d, void *cuda_stream, float *dev_scores_out,
                                       unsigned *dev_flags_out) {
  return step_replicas(h, host_dev_xs, kind, 0u, B, T, d, cuda_stream, dev_scores_out, dev_flags_out, true);
}

int sentinel_replace_if_flagged(sentinel_verifier *h, void *dev_x_inout, sentinel_kind kind, int B, int T,
                                int d, int fill, void *cuda_stream, unsigned *dev_replaced_out) {
  int rc = check_call(h, dev_x_inout, kind, B, T, d);
  if (rc) return rc;
  if (fill != 0 && fill != 1) return fail(h, SENTINEL_ERR_INVALID_ARG, "fill must be 0 (reference) or 1 (zeros), got %d", fill);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  int sms = 0;
  SENTINEL_CUDA(h, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->cfg.device));
  const long long n_chunks = (long long)(h->N / 8);
  long long grid = (long long)sms * 8;                       // 2048 threads per SM, grid-stride
  const long long need = (n_chunks + kReplaceThreads - 1) / kReplaceThreads;
  if (grid > need) grid = need;
  replace_kernel<<<(unsigned)grid, kReplaceThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      h->hs, (int)kind, h->ema[kind][0], h->ema[kind][1], h->bf16 ? 1 : 0, static_cast<uint16_t *>(dev_x_inout), n_chunks,
      h->chan_ref ? (long long)(h->cfg.d / 8) : h->shared_ref ? (long long)(h->ema_elems / 8) : 0ll,
      h->chan_per_sample ? (long long)(h->Ns / 8) : 0ll, fill,
      dev_replaced_out);
  SENTINEL_CUDA(h, cudaGetLastError());
  return SENTINEL_OK;
}

int sentinel_set_directions(sentinel_verifier *h, const void *dev_u_bf16, int L, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!dev_u_bf16) return fail(h, SENTINEL_ERR_INVALID_ARG, "u is NULL");
  if (h->started) return fail(h, SENTINEL_ERR_INVALID_ARG, "the metric set is fixed once a step was taken or a state imported");
  if (h->shared_ref || h->chan_ref) return fail(h, SENTINEL_ERR_UNSUPPORTED, "the sliced Wasserstein chain reads a [B,T,d] reference: not available with ref_over_batch");
  if (h->cfg.d % 8 != 0) return fail(h, SENTINEL_ERR_UNALIGNED, "d = %d is not a multiple of 8", h->cfg.d);
  int rc = check_swd_shape(h, L, h->cfg.T, h->cfg.d);
  if (rc) return rc;
  const size_t smem = refresh_smem_doubles(h->cap0, h->cap1, h->units0, h->units1, kNumMetrics) * sizeof(double);
  if (smem > 200u * 1024u)
    return fail(h, SENTINEL_ERR_UNSUPPORTED, "with four metrics the windows' working copies need %zu bytes of shared memory, 204800 are available", smem);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t u_bytes = (size_t)L * h->cfg.d * sizeof(uint16_t);
  uint16_t *u = nullptr;
  float *scratch = nullptr, *out = nullptr;
  cudaError_t e = cudaMalloc((void **)&u, u_bytes);
  if (e == cudaSuccess) e = cudaMalloc((void **)&scratch, swd_scratch_floats(L, h->cfg.B, h->cfg.T) * sizeof(float));
  const size_t out_floats = (size_t)h->R * (1 + h->cfg.B);      // a block of 1+B per worker
  if (e == cudaSuccess) e = cudaMalloc((void **)&out, out_floats * sizeof(float));
  // the reference's own projections, per kind, current and spare: m_0 = 0 projects to 0
  const size_t pm_bytes = (size_t)h->cfg.B * h->cfg.T * L * sizeof(double);
  double *pm[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};
  for (int k = 0; k < 2; ++k)
    for (int j = 0; j < 2; ++j) {
      if (e == cudaSuccess) e = cudaMalloc((void **)&pm[k][j], pm_bytes);
      if (e == cudaSuccess) e = cudaMemsetAsync(pm[k][j], 0, pm_bytes, s);
    }
  if (e == cudaSuccess) e = cudaMemcpyAsync(u, dev_u_bf16, u_bytes, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(out, 0, out_floats * sizeof(float), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    cudaFree(u); cudaFree(scratch); cudaFree(out);
    for (int k = 0; k < 2; ++k)
      for (int j = 0; j < 2; ++j) cudaFree(pm[k][j]);
    return fail(h, SENTINEL_ERR_CUDA, "setting the directions failed: %s", cudaGetErrorString(e));
  }
  cudaFree(h->sw_u); cudaFree(h->sw_scratch); cudaFree(h->sw_out);   // directions set twice before the first step
  for (int k = 0; k < 2; ++k)
    for (int j = 0; j < 2; ++j) {
      cudaFree(h->sw_pm[k][j]);
      h->sw_pm[k][j] = pm[k][j];
    }
  h->sw_pm_valid[0] = h->sw_pm_valid[1] = true;
  h->sw_u = u; h->sw_scratch = scratch; h->sw_out = out;
  h->sw_L = L;
  h->n_metrics = kNumMetrics;
  h->refresh_smem = smem;
  return SENTINEL_OK;
}

int sentinel_num_metrics(const sentinel_verifier *h) { return h ? h->n_metrics : 0; }

int sentinel_sliced_wasserstein(const void *dev_x, const float *dev_m, const void *dev_u_bf16, int L, int B,
                                int T, int d, int device, void *cuda_stream, float *dev_sw_out) {
  if (!dev_x || !dev_m || !dev_u_bf16 || !dev_sw_out) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "x, m, u or sw_out is NULL");
  int rc = check_shape(nullptr, B, T, d);
  if (rc) return rc;
  if (!aligned16(dev_x) || !aligned16(dev_m) || !aligned16(dev_u_bf16)) return fail(nullptr, SENTINEL_ERR_UNALIGNED, "x, m or u is not 16-byte aligned");
  rc = check_swd_shape(nullptr, L, T, d);
  if (rc) return rc;
  int ndev = 0;
  SENTINEL_CUDA(nullptr, cudaGetDeviceCount(&ndev));
  if (device < 0 || device >= ndev) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "device %d does not exist", device);
  DeviceGuard guard(device);
  SENTINEL_CUDA(nullptr, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int sms = 0;
  SENTINEL_CUDA(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));

  float *scratch = nullptr;
  keep_pool_warm(device);
  SENTINEL_CUDA(nullptr, cudaMallocAsync((void **)&scratch, swd_scratch_floats(L, B, T) * sizeof(float), s));
  cudaError_t e = run_swd(static_cast<const uint16_t *>(dev_x), dev_m, nullptr, false, nullptr, nullptr,
                          static_cast<const uint16_t *>(dev_u_bf16), L, B, T, d, sms, scratch, dev_sw_out,
                          ProjectionState(), s);
  cudaError_t fe = cudaFreeAsync(scratch, s);
  SENTINEL_CUDA(nullptr, e);
  SENTINEL_CUDA(nullptr, fe);
  return SENTINEL_OK;
}

int sentinel_get_stats(sentinel_verifier *h, sentinel_kind kind, float *dev_stats_out, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!dev_stats_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "stats_out is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "bad kind %d", (int)kind);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  SENTINEL_CUDA(h, cudaMemcpyAsync(dev_stats_out, h->stats[kind], (size_t)(1 + h->cfg.B) * kNumStats * sizeof(float),
                                   cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
  return SENTINEL_OK;
}

int sentinel_get_thresholds(sentinel_verifier *h, sentinel_kind kind, double *host_out, int *host_valid, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "host_out is NULL");
  if (kind != SENTINEL_ACT && kind != SENTINEL_GRAD) return fail(h, SENTINEL_ERR_INVALID_ARG, "bad kind %d", (int)kind);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int rc = run_refresh(h, s);
  if (rc) return rc;
  HandleState snap;
  SENTINEL_CUDA(h, cudaMemcpyAsync(&snap, h->hs, sizeof snap, cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));
  for (int L = 0; L < 2; ++L)                     // packed to the metrics in use
    for (int i = 0; i < h->n_metrics; ++i) {
      memcpy(host_out + ((size_t)L * h->n_metrics + i) * kNumThr, snap.kind[kind].thr[L][i], kNumThr * sizeof(double));
      if (host_valid) host_valid[L * h->n_metrics + i] = snap.kind[kind].has_thr[L][i];
    }
  return SENTINEL_OK;
}

int sentinel_get_counters(sentinel_verifier *h, long long *host_out, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "host_out is NULL");
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  HandleState snap;
  SENTINEL_CUDA(h, cudaMemcpyAsync(&snap, h->hs, sizeof snap, cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));
  host_out[0] = snap.violations[0];
  host_out[1] = snap.clean_streak[0];
  host_out[2] = snap.banned[0];
  host_out[3] = snap.kind[0].steps;
  host_out[4] = snap.kind[1].steps;
  host_out[5] = snap.error;
  return SENTINEL_OK;
}

int sentinel_set_token_stats_buffer(sentinel_verifier *h, float *dev_buf) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (dev_buf && !aligned16(dev_buf)) return fail(h, SENTINEL_ERR_UNALIGNED, "token buffer is not 16-byte aligned");
  if (dev_buf && (h->shared_ref || h->chan_ref)) return fail(h, SENTINEL_ERR_UNSUPPORTED, "per-token sums are not written with a [T,d] or [d] reference");
  const int tpr = tiles_per_row(h->cfg.d);
  if (dev_buf && tpr > 1 && !h->token_part) {      // rows of several tiles need a place for the shares
    DeviceGuard guard(h->cfg.device);
    SENTINEL_CUDA(h, guard.status);
    SENTINEL_CUDA(h, cudaMalloc((void **)&h->token_part, (size_t)h->cfg.B * h->cfg.T * tpr * 4 * sizeof(float)));
  }
  h->token_buf = dev_buf;
  return SENTINEL_OK;
}

int sentinel_get_worker_counters(sentinel_verifier *h, int worker, long long *host_out, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_out) return fail(h, SENTINEL_ERR_INVALID_ARG, "host_out is NULL");
  if (worker < 0 || worker >= h->R) return fail(h, SENTINEL_ERR_INVALID_ARG, "worker %d is outside 0..%d", worker, h->R - 1);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  HandleState snap;
  SENTINEL_CUDA(h, cudaMemcpyAsync(&snap, h->hs, sizeof snap, cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));
  host_out[0] = snap.violations[worker];
  host_out[1] = snap.clean_streak[worker];
  host_out[2] = snap.banned[worker];
  return SENTINEL_OK;
}

int sentinel_reset_worker(sentinel_verifier *h, int worker, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (worker < 0 || worker >= h->R) return fail(h, SENTINEL_ERR_INVALID_ARG, "worker %d is outside 0..%d", worker, h->R - 1);
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  reset_worker_kernel<<<1, 1, 0, static_cast<cudaStream_t>(cuda_stream)>>>(h->hs, worker);
  SENTINEL_CUDA(h, cudaGetLastError());
  return SENTINEL_OK;
}

size_t sentinel_state_bytes(const sentinel_verifier *h) {
  if (!h) return 0;
  return kHeaderBytes + sizeof(BlobWorkers) + 2 * kind_blob_bytes(h);
}

int sentinel_export_state(sentinel_verifier *h, void *host_buf, size_t n, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_buf) return fail(h, SENTINEL_ERR_INVALID_ARG, "host_buf is NULL");
  if (n < sentinel_state_bytes(h)) return fail(h, SENTINEL_ERR_STATE_SIZE, "buffer of %zu bytes, %zu needed", n, sentinel_state_bytes(h));
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int rc = run_refresh(h, s);
  if (rc) return rc;
  HandleState snap;
  SENTINEL_CUDA(h, cudaMemcpyAsync(&snap, h->hs, sizeof snap, cudaMemcpyDeviceToHost, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));

  unsigned char *out = static_cast<unsigned char *>(host_buf);
  memset(out, 0, kHeaderBytes);
  BlobHeader hd = {kMagic, kVersion, h->cfg.B, h->cfg.T, h->cfg.d, h->cfg.window_steps, h->R, h->n_metrics, h->chan_per_sample ? 3 : h->chan_ref ? 2 : h->shared_ref ? 1 : 0};
  memcpy(out, &hd, sizeof hd);
  out += kHeaderBytes;
  BlobWorkers bw;
  memcpy(bw.violations, snap.violations, sizeof bw.violations);
  memcpy(bw.clean_streak, snap.clean_streak, sizeof bw.clean_streak);
  memcpy(bw.banned, snap.banned, sizeof bw.banned);
  memcpy(out, &bw, sizeof bw);
  out += sizeof bw;
  std::vector<double> ring(ring_doubles(h));
  for (int k = 0; k < 2; ++k) {
    const KindState &ks = snap.kind[k];
    BlobKindHead kh;
    memset(&kh, 0, sizeof kh);
    kh.steps = ks.steps;
    memcpy(kh.count, ks.hist_count, sizeof kh.count);
    memcpy(kh.valid, ks.has_thr, sizeof kh.valid);
    memcpy(kh.thr, ks.thr, sizeof kh.thr);
    memcpy(out, &kh, sizeof kh);
    out += sizeof kh;
    SENTINEL_CUDA(h, cudaMemcpyAsync(ring.data(), h->hist[k], ring.size() * sizeof(double), cudaMemcpyDeviceToHost, s));
    SENTINEL_CUDA(h, cudaStreamSynchronize(s));
    double *dst = reinterpret_cast<double *>(out);
    for (int L = 0; L < 2; ++L) {                   // unroll each ring, oldest entry first
      const int cap = L ? h->cap1 : h->cap0, size = ring_size(cap, L ? h->units1 : h->units0);
      for (int i = 0; i < kNumMetrics; ++i) {
        const size_t src_off = ring_offset(L, i, h->cap0, h->cap1, h->units0, h->units1);
        for (int j = 0; j < cap; ++j)
          dst[j] = (j < ks.hist_count[L]) ? ring[src_off + (size_t)((ks.hist_head[L] + j) % size)] : 0.0;
        dst += cap;
      }
    }
    out = reinterpret_cast<unsigned char *>(dst);
    if (h->bf16) {                                  // the blob always carries fp32: widen (exact)
      std::vector<uint16_t> half(h->ema_elems);
      SENTINEL_CUDA(h, cudaMemcpyAsync(half.data(), h->ema[k][ks.active], h->ema_bytes, cudaMemcpyDeviceToHost, s));
      SENTINEL_CUDA(h, cudaStreamSynchronize(s));
      for (size_t e = 0; e < h->ema_elems; ++e) {
        const unsigned bits = (unsigned)half[e] << 16;
        memcpy(out + e * sizeof(float), &bits, sizeof bits);
      }
    } else {
      SENTINEL_CUDA(h, cudaMemcpyAsync(out, h->ema[k][ks.active], h->ema_elems * sizeof(float), cudaMemcpyDeviceToHost, s));
      SENTINEL_CUDA(h, cudaStreamSynchronize(s));
    }
    out += h->ema_elems * sizeof(float);
  }
  return SENTINEL_OK;
}

int sentinel_import_state(sentinel_verifier *h, const void *host_buf, size_t n, void *cuda_stream) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  if (!host_buf) return fail(h, SENTINEL_ERR_INVALID_ARG, "host_buf is NULL");
  if (n < sentinel_state_bytes(h)) return fail(h, SENTINEL_ERR_STATE_SIZE, "blob of %zu bytes, %zu needed", n, sentinel_state_bytes(h));
  const unsigned char *in = static_cast<const unsigned char *>(host_buf);
  BlobHeader hd;
  memcpy(&hd, in, sizeof hd);
  if (hd.magic != kMagic || hd.version != kVersion)
    return fail(h, SENTINEL_ERR_STATE_SIZE, "not a sentinel state blob of version %u", kVersion);
  if (hd.B != h->cfg.B || hd.T != h->cfg.T || hd.d != h->cfg.d || hd.window_steps != h->cfg.window_steps || hd.n_workers != h->R)
    return fail(h, SENTINEL_ERR_STATE_SIZE, "blob is for shape [%d,%d,%d], window %d, %d workers", hd.B, hd.T, hd.d, hd.window_steps, hd.n_workers);
  if (hd.ref_over_batch != (h->chan_per_sample ? 3 : h->chan_ref ? 2 : h->shared_ref ? 1 : 0))
    return fail(h, SENTINEL_ERR_STATE_SIZE, "blob and verifier differ in the shape of the reference ([B,T,d], [T,d], [d] or [B,d])");
  if (hd.n_metrics != h->n_metrics)
    return fail(h, SENTINEL_ERR_STATE_SIZE, "blob holds %d metrics, this verifier uses %d (set the directions before importing)", hd.n_metrics, h->n_metrics);
  // validate both kinds before touching the device
  const unsigned char *p = in + kHeaderBytes + sizeof(BlobWorkers);
  for (int k = 0; k < 2; ++k) {
    BlobKindHead kh;
    memcpy(&kh, p, sizeof kh);
    if (kh.count[0] < 0 || kh.count[0] > h->cap0 || kh.count[1] < 0 || kh.count[1] > h->cap1)
      return fail(h, SENTINEL_ERR_STATE_SIZE, "history counts in the blob are out of range");
    p += kind_blob_bytes(h);
  }
  DeviceGuard guard(h->cfg.device);
  SENTINEL_CUDA(h, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

  h->started = true;
  h->sw_pm_valid[0] = h->sw_pm_valid[1] = false;   // the next step recomputes the reference's projections from m
  HandleState st;
  memset(&st, 0, sizeof st);
  BlobWorkers bw;
  memcpy(&bw, in + kHeaderBytes, sizeof bw);
  memcpy(st.violations, bw.violations, sizeof bw.violations);
  memcpy(st.clean_streak, bw.clean_streak, sizeof bw.clean_streak);
  memcpy(st.banned, bw.banned, sizeof bw.banned);
  p = in + kHeaderBytes + sizeof(BlobWorkers);
  for (int k = 0; k < 2; ++k) {
    BlobKindHead kh;
    memcpy(&kh, p, sizeof kh);
    p += sizeof kh;
    KindState &ks = st.kind[k];
    ks.steps = kh.steps;
    ks.active = 0;
    ks.refresh_pending = 0;
    memcpy(ks.hist_count, kh.count, sizeof kh.count);
    ks.hist_head[0] = ks.hist_head[1] = 0;
    memcpy(ks.has_thr, kh.valid, sizeof kh.valid);
    memcpy(ks.thr, kh.thr, sizeof kh.thr);
    ks.last_joined[0] = ks.last_joined[1] = 0;
    ks.last_evicted[0] = ks.last_evicted[1] = 0;
    {   // windows start at ring slot 0; the ascending copies are sorted here, on the host
      std::vector<double> rings(ring_doubles(h), 0.0), asc(hist_doubles(h), 0.0);
      const double *src = reinterpret_cast<const double *>(p);
      for (int L = 0; L < 2; ++L) {
        const int cap = L ? h->cap1 : h->cap0;
        for (int i = 0; i < kNumMetrics; ++i) {
          double *r = rings.data() + ring_offset(L, i, h->cap0, h->cap1, h->units0, h->units1);
          double *a = asc.data() + sorted_offset(L, i, h->cap0, h->cap1);
          std::copy(src, src + kh.count[L], r);
          std::copy(src, src + kh.count[L], a);
          std::sort(a, a + kh.count[L]);
          src += cap;
        }
      }
      SENTINEL_CUDA(h, cudaMemcpyAsync(h->hist[k], rings.data(), rings.size() * sizeof(double), cudaMemcpyHostToDevice, s));
      SENTINEL_CUDA(h, cudaMemcpyAsync(h->sorted[k], asc.data(), asc.size() * sizeof(double), cudaMemcpyHostToDevice, s));
      SENTINEL_CUDA(h, cudaStreamSynchronize(s));     // the staging vectors go out of scope
    }
    p += hist_doubles(h) * sizeof(double);
    if (h->bf16) {                                  // narrow, to nearest even (exact for a bf16 verifier's own blob)
      std::vector<uint16_t> half(h->ema_elems);
      for (size_t e = 0; e < h->ema_elems; ++e) {
        unsigned bits;
        memcpy(&bits, p + e * sizeof(float), sizeof bits);
        if ((bits & 0x7F800000u) != 0x7F800000u) bits += 0x7FFFu + ((bits >> 16) & 1u);
        half[e] = (uint16_t)(bits >> 16);
      }
      SENTINEL_CUDA(h, cudaMemcpyAsync(h->ema[k][0], half.data(), h->ema_bytes, cudaMemcpyHostToDevice, s));
      SENTINEL_CUDA(h, cudaStreamSynchronize(s));     // the staging vector goes out of scope
    } else {
      SENTINEL_CUDA(h, cudaMemcpyAsync(h->ema[k][0], p, h->ema_elems * sizeof(float), cudaMemcpyHostToDevice, s));
    }
    p += h->ema_elems * sizeof(float);
  }
  SENTINEL_CUDA(h, cudaMemcpyAsync(h->hs, &st, sizeof st, cudaMemcpyHostToDevice, s));
  SENTINEL_CUDA(h, cudaStreamSynchronize(s));
  return SENTINEL_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// sentinel_distance_noalloc: the stateless distance with its scratch in the library image

namespace {

// Scratch of the no-allocation entry point.  In host code this name is only a stand-in for the
// symbol: the address a kernel may use is looked up per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SENTINEL_NOALLOC_SCRATCH_BYTES];

constexpr int kNoAllocMaxDevices = 64;
constexpr size_t kNoAllocTicketBytes = 256;          // the ticket word, kept on its own 256 bytes
std::mutex g_noalloc_mutex;
unsigned char *g_noalloc_addr[kNoAllocMaxDevices];  // device address of the array, per device

// Resolves the array's address on `device` (which must be current).  Once per device.
cudaError_t noalloc_scratch_address(int device, unsigned char **out) {
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_addr[device]) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_addr[device] = static_cast<unsigned char *>(p);
  }
  *out = g_noalloc_addr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" {

int sentinel_distance_noalloc(const void *dev_x, const float *dev_m, int B, int T, int d, int device,
                              void *cuda_stream, float *dev_scores_out, float *dev_stats_out) {
  if (!dev_x || !dev_m || !dev_scores_out) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "x, m or scores_out is NULL");
  int rc = check_shape(nullptr, B, T, d);
  if (rc) return rc;
  if (!aligned16(dev_x) || !aligned16(dev_m)) return fail(nullptr, SENTINEL_ERR_UNALIGNED, "x or m is not 16-byte aligned");
  int ndev = 0;
  SENTINEL_CUDA(nullptr, cudaGetDeviceCount(&ndev));
  if (device < 0 || device >= ndev || device >= kNoAllocMaxDevices)
    return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "device %d does not exist or is beyond the %d this entry point tracks", device, kNoAllocMaxDevices);
  DeviceGuard guard(device);
  SENTINEL_CUDA(nullptr, guard.status);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

  std::string oerr;
  const int G = distance_ctas(device, B, T, &oerr);
  if (G < 1) return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "%s", oerr.c_str());
  const size_t slot_bytes = (size_t)G * kSegsPerCta * kSlotWords * sizeof(unsigned long long);
  if (slot_bytes + kNoAllocTicketBytes > (size_t)SENTINEL_NOALLOC_SCRATCH_BYTES)
    return fail(nullptr, SENTINEL_ERR_UNSUPPORTED,
                "this launch needs %zu bytes of scratch (%d streaming CTAs), the built-in array holds %d",
                slot_bytes + kNoAllocTicketBytes, G, SENTINEL_NOALLOC_SCRATCH_BYTES);

  unsigned char *scratch = nullptr;
  SENTINEL_CUDA(nullptr, noalloc_scratch_address(device, &scratch));
  // layout: [ticket: 256 bytes][slots]; the slots are rewritten by every launch, the ticket
  // must start at zero whatever an earlier call left there
  SENTINEL_CUDA(nullptr, cudaMemsetAsync(scratch, 0, kNoAllocTicketBytes, s));

  StreamArgs a;
  memset(&a, 0, sizeof a);
  a.x = static_cast<const uint16_t *>(dev_x);
  a.m_ext = dev_m;
  a.partials = reinterpret_cast<unsigned long long *>(scratch + kNoAllocTicketBytes);
  a.ticket = reinterpret_cast<unsigned *>(scratch);
  a.scores_out = dev_scores_out;
  a.stats_out = dev_stats_out;
  a.B = B; a.T = T; a.d = d; a.G = G;
  a.x_row_stride = d;
  a.x_extent = a.ref_extent = (long long)B * T * d;
  a.partials_words = (long long)G * kSegsPerCta * kSlotWords;
  a.n_metrics = 3;
  a.mode = kModeDistance;
  stream_kernel_t<false, false><<<G + 1, kThreads, 0, s>>>(a);
  SENTINEL_CUDA(nullptr, cudaGetLastError());
  return SENTINEL_OK;
}

int sentinel_bounds_violations(int device, unsigned long long *host_count, int *host_first_site) {
  if (!host_count) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "host_count is NULL");
#ifdef SENTINEL_CHECK_BOUNDS
  int ndev = 0;
  SENTINEL_CUDA(nullptr, cudaGetDeviceCount(&ndev));
  if (device < 0 || device >= ndev) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "device %d does not exist", device);
  DeviceGuard guard(device);
  SENTINEL_CUDA(nullptr, guard.status);
  SENTINEL_CUDA(nullptr, cudaDeviceSynchronize());
  int site = 0;
  SENTINEL_CUDA(nullptr, cudaMemcpyFromSymbol(host_count, g_bounds_violations, sizeof *host_count));
  SENTINEL_CUDA(nullptr, cudaMemcpyFromSymbol(&site, g_bounds_first_site, sizeof site));
  if (host_first_site) *host_first_site = site;
  return SENTINEL_OK;
#else
  (void)device;
  *host_count = 0ull;
  if (host_first_site) *host_first_site = 0;
  return fail(nullptr, SENTINEL_ERR_UNSUPPORTED, "this library was built without bounds checks (-DSENTINEL_CHECK_BOUNDS)");
#endif
}

const char *sentinel_last_error(const sentinel_verifier *h) { return h ? h->err.c_str() : g_error.c_str(); }

int sentinel_destroy(sentinel_verifier *h) {
  if (!h) return fail(nullptr, SENTINEL_ERR_INVALID_ARG, "handle is NULL");
  DeviceGuard guard(h->cfg.device);
  cudaError_t e = guard.status;
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  free_all(h);
  delete h;
  if (e != cudaSuccess) return fail(nullptr, SENTINEL_ERR_CUDA, "destroy: %s", cudaGetErrorString(e));
  return SENTINEL_OK;
}

}  // extern "C"
