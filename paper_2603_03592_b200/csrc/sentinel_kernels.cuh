// Device code of libsentinel: one streaming pass over a [B,T,d] bf16 tensor x and the fp32
// reference m that (1) accumulates, per sample, the sufficient statistics of the paper's
// distance measures (Sec. 3.1), (2) writes the EMA candidate beta*m + (1-beta)*x (Eq. 1) into
// the spare reference buffer, and (3) in the last CTA to finish, turns the sums into scores,
// applies the Tukey test (Eq. 3), keeps the violation counter, appends to the history and
// commits the candidate by flipping the active-buffer index.  Thresholds (Alg. 5) for the next
// step are recomputed by CTA 0 of the *next* launch while the other CTAs stream.
//
// sm_100a only: 256-bit global loads/stores (ld/st.global.v8.f32).
#pragma once

#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include <type_traits>

namespace sentinel {

constexpr int kNumMetrics = 4;          // room for L1, z-scored L2, sign flips and the sliced Wasserstein
                                        // distance; a launch uses the first n_metrics (3 or 4) of them
constexpr int kNumStats = 8;
constexpr int kNumThr = 6;
constexpr int kMaxB = 64;
constexpr int kMaxWindow = 4096;
constexpr int kThreads = 640;             // threads per CTA: with kUnroll = 2 about 60 KB of loads
                                          // in flight per SM, where the read/write mix peaked in sweeps
constexpr int kWarps = kThreads / 32;
constexpr int kSlotWords = 8;             // 64-bit words per partial slot
constexpr int kUnroll = 2;                // 8-element chunks per lane per loop trip
constexpr int kUnrollBf16 = 4;            // the same with a bf16 reference (vector rows)

constexpr int kMaxWorkers = 16;           // workers (replicas of a stage) one handle can follow

// single submission (stream_kernel_t): verify / warm-up / stateless distance; all workers of a
// stage in one launch (replica_kernel): verify / warm-up, passed to each worker's finalize pass
enum Mode : int { kModeVerify = 0, kModeWarmup = 1, kModeDistance = 2,
                  kModeReplicaVerify = 3, kModeReplicaWarmup = 4 };

// flag bits (mirrors the public header)
constexpr unsigned kFlagNonfinite = 1u << 7;
constexpr unsigned kFlagCommitted = 1u << 16;
constexpr unsigned kFlagSevere = 1u << 17;
constexpr unsigned kFlagBanned = 1u << 18;
constexpr unsigned kFlagNoThresholds = 1u << 19;
constexpr unsigned kFlagNaturalShift = 1u << 20;
constexpr unsigned kFlagTaintedElsewhere = 1u << 21;

// word 7 of a partial slot: bits 0-2 flags, bits 8-15 tag (1 + sample index, 0 = slot unused),
// bits 16-31 the sample's first x (bf16 bits), bits 32-63 the sample's first m (fp32 bits)
constexpr unsigned long long kBitNonfinite = 1ull, kBitXVaries = 2ull, kBitMVaries = 4ull;
constexpr int kTagShift = 8, kX0Shift = 16, kM0Shift = 32;

struct Alg5Params {
  double alpha, gamma_g, gamma_s, lambda, eps, shrink_ratio;
  int n_max;
  int pad;
};

// Device-resident state of one kind (activations or gradients) of one boundary.
struct KindState {
  long long steps;
  int active;             // which of the two EMA buffers holds m_{t-1}
  int refresh_pending;    // Alg. 5 is owed for the history as it stands
  int hist_count[2];      // entries in the window, per level
  int hist_head[2];       // ring position of the oldest entry
  int last_joined[2];     // entries the last step appended / pushed out, per level: what the
  int last_evicted[2];    //   pending refresh has to merge into the sorted copy
  int last_flagged;       // the last verified step of this kind raised a flag (no commit)
  unsigned step_collected;  // multi-worker iteration in progress: workers scored so far,
  unsigned step_tainted;    //   workers that raised a flag,
  unsigned step_nonfinite;  //   workers whose tensor held a NaN or an infinity,
  unsigned step_elsewhere;  //   workers tainted at another stage (not collected)
  int commit_pending;     // [d] reference: the step committed; channel_mean_kernel writes the candidate and flips `active`
  long long mean_done_step; // the iteration whose mean over the workers is already in place
  int has_thr[2][kNumMetrics];
  double thr[2][kNumMetrics][kNumThr];   // q1 q2 q3 k tau_lower tau_upper
};

struct HandleState {
  int error;
  unsigned ticket;
  unsigned ticket2;       // the ticket of channel_mean_kernel
  int pad;
  int violations[kMaxWorkers], clean_streak[kMaxWorkers], banned[kMaxWorkers];   // per worker
  KindState kind[2];
};

struct StreamArgs {
  const uint16_t *x;               // bf16 [B,T,d]
  const float *m_ext;              // distance mode: caller's reference; else unused
  void *ema[2];                    // the two reference buffers of this kind: fp32, or bf16 if ema_bf16
  HandleState *hs;                 // nullptr in distance mode
  double *hist;                    // this kind's rings: level 0 [4][cap0+units0], level 1 [4][cap1+units1]
  double *sorted;                  // the same windows kept ascending: [4][cap0], [4][cap1]
  unsigned long long *partials;    // [G][2][kSlotWords]
  unsigned *ticket;
  float *scores_out;               // [(1+B)*n_metrics] or nullptr
  unsigned *flags_out;             // [1+B] or nullptr
  float *stats_out;                // [(1+B)*8] or nullptr
  float *token_out;                // [B,T,4] or nullptr
  float *token_part;               // [B*T][tiles per row][4]: per-tile shares when a row has several tiles
  int B, T, d;
  int G;                           // streaming CTAs (the grid has one more)
  int mode, kind;
  float beta, one_minus_beta;
  int cap0, cap1;
  int units0, units1;              // entries one iteration can append per level: R and R*B
  int R;                           // workers of the stage
  int ema_bf16;                    // the reference is stored as bf16 (single submissions only)
  long long x_row_stride;          // elements from one row of x to the next (d when dense)
  const float *sw;                 // [1+B] sliced Wasserstein distance of every unit, computed by the
                                   // launches before this one; nullptr when n_metrics = 3
  int n_metrics;                   // metrics in use: 3, or 4 with the sliced Wasserstein distance
  int ref_per_sample;              // reduced reference with a vector per sample ([B,d]) instead of one ([d])
  Alg5Params a5;
  double severe_mult;
  int ban_violations, forgiveness_steps;
  unsigned metric_mask;
  int defer_commit;                // [d] reference: the commit is carried out by channel_mean_kernel
  float *col_part;                 // [d] reference: column sums of x, [G][2][channel_slots(d)][512]
  // extents, in elements, of what the indices below are checked against in the checked build
  long long x_extent;              // of x from its first element: (B*T - 1) * row stride + d
  long long ref_extent;            // of one reference buffer
  long long partials_words;        // of the partial slots
  long long ring_doubles, sorted_doubles;   // of this kind's rings and ascending copies
  long long col_floats;            // of col_part
};

// ---------------------------------------------------------------------------------------------
// The checked build (-DSENTINEL_CHECK_BOUNDS, a second library target): before a kernel touches
// global memory through an index that was worked out from the shape (B, T, d, the row stride, the
// number of CTAs, the ring sizes), the range is compared with the extent of the buffer.  An access
// that would leave it is skipped and counted; nothing traps.  The count and the site of the first
// violation are read with sentinel_bounds_violations(), and the last CTA of a launch writes
// kErrBounds into HandleState.error.  In the normal build the checks compile to nothing.
constexpr int kErrBounds = 2;                     // HandleState.error: an index left its buffer (checked build)
enum Site : int { kSiteX = 1, kSiteRefIn, kSiteRefOut, kSiteToken, kSiteSlot, kSiteRing, kSiteSorted, kSiteOut,
                  kSiteStageX, kSiteStageRef, kSiteColumns, kSiteReplace, kSiteSwdLists, kSiteSwdPartial };
#ifdef SENTINEL_CHECK_BOUNDS
__device__ unsigned long long g_bounds_violations = 0ull;
__device__ int g_bounds_first_site = 0;
__device__ __forceinline__ bool in_bounds(int site, long long first, long long count, long long extent) {
  if (first >= 0 && count >= 0 && first + count <= extent) return true;
  atomicAdd(&g_bounds_violations, 1ull);
  atomicCAS(&g_bounds_first_site, 0, site);
  return false;
}
#define SENTINEL_BOUNDS(site, first, count, extent) \
  ::sentinel::in_bounds((site), (long long)(first), (long long)(count), (long long)(extent))
#else
#define SENTINEL_BOUNDS(site, first, count, extent) true
#endif

// ---------------------------------------------------------------------------------------------
// memory access helpers

struct __align__(32) F8 { float v[8]; };

__device__ __forceinline__ uint4 ld_x128(const uint16_t *p) {
  uint4 r;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
      : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ F8 ld_m256(const float *p) {
  F8 r;
  asm("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
      : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]),
        "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7]) : "l"(p));
  return r;
}
__device__ __forceinline__ void st_m256(float *p, const F8 &r) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]),
                  "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7]) : "memory");
}

// The reference as the kernels see it: 8 consecutive elements as floats, whatever the storage.
// A bf16 reference is widened on load and rounded to nearest even (cvt.rn) on store.
__device__ __forceinline__ unsigned pack_bf16x2_rn(float lo, float hi) {
  unsigned r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));   // upper half <- first operand
  return r;
}
__device__ __forceinline__ F8 widen_bf16x8(const uint4 &v) {
  const unsigned w[4] = {v.x, v.y, v.z, v.w};
  F8 r;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    r.v[2 * j] = __uint_as_float(w[j] << 16);
    r.v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
  return r;
}
template <bool kBf16>
__device__ __forceinline__ F8 load_m8(const void *m, size_t idx) {
  if (kBf16) return widen_bf16x8(ld_x128(static_cast<const uint16_t *>(m) + idx));
  return ld_m256(static_cast<const float *>(m) + idx);
}
template <bool kBf16>
__device__ __forceinline__ void store_m8(void *m, size_t idx, const F8 &r) {
  if (kBf16) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(static_cast<uint16_t *>(m) + idx), "r"(pack_bf16x2_rn(r.v[0], r.v[1])),
                    "r"(pack_bf16x2_rn(r.v[2], r.v[3])), "r"(pack_bf16x2_rn(r.v[4], r.v[5])),
                    "r"(pack_bf16x2_rn(r.v[6], r.v[7])) : "memory");
  } else {
    st_m256(static_cast<float *>(m) + idx, r);
  }
}
template <bool kBf16>
__device__ __forceinline__ float load_m1(const void *m, size_t idx) {
  if (kBf16) return __uint_as_float((unsigned)static_cast<const uint16_t *>(m)[idx] << 16);
  return static_cast<const float *>(m)[idx];
}
template <bool kBf16>
__device__ __forceinline__ void store_m1(void *m, size_t idx, float v) {
  if (kBf16) static_cast<uint16_t *>(m)[idx] = (uint16_t)(pack_bf16x2_rn(v, 0.f) & 0xFFFFu);
  else static_cast<float *>(m)[idx] = v;
}

// ---------------------------------------------------------------------------------------------
// staging through shared memory: bulk asynchronous copies that complete on an mbarrier
//
// A warp fills its own stages (one lane issues the copies) and is the only one to wait on them.
// A wait that does not end -- it always should -- gives up after kStageWaitNs; the kernel then
// records kErrStagingTimeout in HandleState.error and leaves the affected rows out.
constexpr int kTileBytesM = 32 * kUnroll * 8 * 4; // a warp tile (512 elements) of an fp32 reference: 2048 bytes
constexpr int kTileBytesX = 32 * kUnroll * 8 * 2; // and of a bf16 tensor: 1024 bytes
constexpr unsigned long long kStageWaitNs = 2000000000ull;
constexpr int kErrStagingTimeout = 1;             // HandleState.error: a staged copy did not arrive

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned arrivals) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
// global -> this CTA's shared memory, 16-byte aligned on both sides, a multiple of 16 bytes
__device__ __forceinline__ void bulk_copy_in(unsigned dst, const void *src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
  unsigned done;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done != 0u;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Waits for the phase `parity` of a stage's barrier; false if it did not complete in kStageWaitNs.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > kStageWaitNs) return false;
  }
}

// ---------------------------------------------------------------------------------------------
// sign mismatches on packed bf16 pairs
//
// With the sign bits of the two m's of a pair at bits 15 and 31 of `msp`, (w ^ msp) & 0x80008000
// has a bit set per element of the pair whose sign bit differs from m's, and a byte-wise dot
// product with ones adds them up, 0x80 = kFlipUnit each.  That is the count of sign(x) != sign(m)
// as long as neither side holds an exact zero (a zero differs from any non-zero whatever its sign
// bit): the caller makes sure of m beforehand and follows the smallest magnitude of x with
// min_abs_bf16x2 to correct the count of a tile in which it reached zero.
constexpr unsigned kFlipUnit = 128u;

__device__ __forceinline__ unsigned min_abs_bf16x2(unsigned a, unsigned b) {   // per half: min(|a|, |b|), sign bit unspecified
  unsigned r;
  asm("min.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// ---------------------------------------------------------------------------------------------
// two single-precision operations per instruction (add/sub/fma.f32x2, new on sm_100): the
// arithmetic-bound kernels below issue half as many floating-point instructions with them; each
// half is rounded as the scalar instruction would round it
struct F2 { float lo, hi; };
__device__ __forceinline__ F2 add2(F2 a, F2 b) {
  F2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tadd.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.lo), "=f"(r.hi) : "f"(a.lo), "f"(a.hi), "f"(b.lo), "f"(b.hi));
  return r;
}
__device__ __forceinline__ F2 sub2(F2 a, F2 b) {
  F2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tsub.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.lo), "=f"(r.hi) : "f"(a.lo), "f"(a.hi), "f"(b.lo), "f"(b.hi));
  return r;
}
__device__ __forceinline__ F2 mul2(F2 a, F2 b) {
  F2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.lo), "=f"(r.hi) : "f"(a.lo), "f"(a.hi), "f"(b.lo), "f"(b.hi));
  return r;
}
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) {
  F2 r;
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\tfma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.lo), "=f"(r.hi) : "f"(a.lo), "f"(a.hi), "f"(b.lo), "f"(b.hi), "f"(c.lo), "f"(c.hi));
  return r;
}

// ---------------------------------------------------------------------------------------------
// per-element work

struct GroupAcc {            // fp32 partial sums over one loop trip (<= 8*kUnroll elements)
  float sx, sxx, sm, smm, sxm, ab;
  unsigned flips;
};

// First and second moments are accumulated on x - x0 and m - m0, where x0 / m0 is the first
// element of the sample: variance and covariance do not depend on the shift, and the shifted
// values are of the size of the spread, so a mean far from zero costs no digits.
__device__ __forceinline__ void element(float xf, float mf, float x0, float m0, GroupAcc &g) {
  const float xs = xf - x0, ms = mf - m0;
  g.sx += xs;
  g.sxx = fmaf(xs, xs, g.sxx);
  g.sm += ms;
  g.smm = fmaf(ms, ms, g.smm);
  g.sxm = fmaf(xs, ms, g.sxm);
  g.ab += fabsf(xf - mf);
  // sign(x) != sign(m) with sign in {-1,0,+1}: either exactly one of them is zero, or both are
  // non-zero and x carrying the extra sign of m is negative
  const float xt = __uint_as_float(__float_as_uint(xf) ^ (__float_as_uint(mf) & 0x80000000u));
  g.flips += (((xf == 0.f) != (mf == 0.f)) || (xt < 0.f)) ? 1u : 0u;
}

struct ThreadAcc {           // carried over the CTA's rows of one sample
  double sx, sxx, sm, smm, sxm, ab;
  unsigned flips;
  unsigned nf_bits;          // non-zero: a bf16 exponent of all ones was seen
  unsigned x_diff, m_diff;   // non-zero: some element differs bitwise from the sample's first
};

// one 8-element chunk: x as 4 packed bf16 pairs, m as 8 floats; returns the EMA candidate in m
__device__ __forceinline__ void chunk(const uint4 &xv, F8 &mv, GroupAcc &g, ThreadAcc &t,
                                      unsigned x0pair, unsigned m0bits, float beta, float omb,
                                      bool write_ema) {
  const float x0 = __uint_as_float(x0pair << 16), m0 = __uint_as_float(m0bits);
  const unsigned w[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    // exponent field 0xFF in either half <=> NaN or infinity
    t.nf_bits |= ((w[j] & 0x7F807F80u) + 0x00800080u) & 0x80008000u;
    t.x_diff |= w[j] ^ x0pair;
    const float x_lo = __uint_as_float(w[j] << 16);
    const float x_hi = __uint_as_float(w[j] & 0xFFFF0000u);
    const float m_lo = mv.v[2 * j], m_hi = mv.v[2 * j + 1];
    t.m_diff |= (__float_as_uint(m_lo) ^ m0bits) | (__float_as_uint(m_hi) ^ m0bits);
    element(x_lo, m_lo, x0, m0, g);
    element(x_hi, m_hi, x0, m0, g);
    if (write_ema) {
      mv.v[2 * j] = fmaf(beta, m_lo, omb * x_lo);
      mv.v[2 * j + 1] = fmaf(beta, m_hi, omb * x_hi);
    }
  }
}

// The same chunk with a bf16 reference, which leaves the arithmetic as the bound (6 bytes per
// element move instead of 10): x and m stay packed pairs as long as they can.  The sums run on
// two-wide instructions (even elements in one half, odd ones in the other; the halves are added
// when the trip is folded), sign mismatches are counted on the packed words (the sign bits of a
// bf16 pair sit where the test wants them), the smallest magnitudes of x and of m are followed so
// that a trip with an exact zero in it can be counted again element by element, and non-finite
// elements show in the sum of |x - m|.  The candidate is fma(beta, m, (1-beta) x) per element,
// each half rounded as the scalar instructions round, then to bf16 (nearest even): bit for bit
// the value of the scalar path.
struct PairAcc {             // one loop trip: two-wide fp32 sums, packed counters
  F2 sx, sxx, sm, smm, sxm;
  float ab[2];
  unsigned flips;            // in units of kFlipUnit
  unsigned zmin;             // per half: smallest magnitude met in x or in m
};

__device__ __forceinline__ void chunk_packed(const uint4 &xv, const uint4 &mraw, uint4 &out, PairAcc &g, ThreadAcc &t,
                                             unsigned x0pair, unsigned m0pair, float x0, float m0, float beta, float omb,
                                             bool write_ema) {
  const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w}, mw[4] = {mraw.x, mraw.y, mraw.z, mraw.w};
  unsigned ow[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    t.x_diff |= xw[j] ^ x0pair;
    t.m_diff |= mw[j] ^ m0pair;
    g.flips = __dp4a((xw[j] ^ mw[j]) & 0x80008000u, 0x01010101u, g.flips);
    g.zmin = min_abs_bf16x2(min_abs_bf16x2(g.zmin, xw[j]), mw[j]);
    const F2 xf = {__uint_as_float(xw[j] << 16), __uint_as_float(xw[j] & 0xFFFF0000u)};
    const F2 mf = {__uint_as_float(mw[j] << 16), __uint_as_float(mw[j] & 0xFFFF0000u)};
    const F2 xs = sub2(xf, F2{x0, x0}), ms = sub2(mf, F2{m0, m0});
    g.sx = add2(g.sx, xs);
    g.sm = add2(g.sm, ms);
    g.sxx = fma2(xs, xs, g.sxx);
    g.smm = fma2(ms, ms, g.smm);
    g.sxm = fma2(xs, ms, g.sxm);
    const F2 df = sub2(xf, mf);
    g.ab[0] += fabsf(df.lo);
    g.ab[1] += fabsf(df.hi);
    if (write_ema) {
      const F2 cand = fma2(F2{beta, beta}, mf, mul2(F2{omb, omb}, xf));
      ow[j] = pack_bf16x2_rn(cand.lo, cand.hi);
    }
  }
  out = make_uint4(ow[0], ow[1], ow[2], ow[3]);
}

// sign(x) != sign(m), three-valued, element by element on a packed chunk (the trips in which the
// packed count does not hold: an exact zero on either side)
__device__ __forceinline__ unsigned flips_exact(const uint4 &xv, const uint4 &mraw) {
  const unsigned xw[4] = {xv.x, xv.y, xv.z, xv.w}, mw[4] = {mraw.x, mraw.y, mraw.z, mraw.w};
  unsigned n = 0u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const unsigned xb = h ? (xw[j] >> 16) : (xw[j] & 0xFFFFu), mb = h ? (mw[j] >> 16) : (mw[j] & 0xFFFFu);
      const bool xz = (xb & 0x7FFFu) == 0u, mz = (mb & 0x7FFFu) == 0u;
      n += ((xz != mz) || (!xz && !mz && ((xb ^ mb) & 0x8000u))) ? 1u : 0u;
    }
  }
  return n;
}
__device__ __forceinline__ unsigned nonfinite_bits(const uint4 &xv) {
  return (((xv.x & 0x7F807F80u) + 0x00800080u) | ((xv.y & 0x7F807F80u) + 0x00800080u) |
          ((xv.z & 0x7F807F80u) + 0x00800080u) | ((xv.w & 0x7F807F80u) + 0x00800080u)) & 0x80008000u;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// A segment's sums, thread -> warp -> CTA in a fixed order (two runs give bit-identical sums),
// written to the segment's slot with the sample's tag and the shift the sums were taken about.
__device__ __forceinline__ void reduce_to_slot(const ThreadAcc &t, int b, unsigned x0, unsigned m0bits,
                                               unsigned long long (*s_part)[kSlotWords], unsigned long long *slot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = (int)blockDim.x >> 5;   // (<= kWarps)
  const double ws[6] = {warp_sum(t.sx), warp_sum(t.sxx), warp_sum(t.sm),
                        warp_sum(t.smm), warp_sum(t.sxm), warp_sum(t.ab)};
  const unsigned long long wf = warp_sum((unsigned long long)t.flips);
  unsigned long long bits = (t.nf_bits ? kBitNonfinite : 0ull) | (t.x_diff ? kBitXVaries : 0ull) |
                            (t.m_diff ? kBitMVaries : 0ull);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
  __syncthreads();                      // s_part may still be read from the previous segment
  if (lane == 0) {
#pragma unroll
    for (int j = 0; j < 6; ++j) s_part[warp][j] = (unsigned long long)__double_as_longlong(ws[j]);
    s_part[warp][6] = wf;
    s_part[warp][7] = bits;
  }
  __syncthreads();
  if (threadIdx.x < kSlotWords) {
    const int j = threadIdx.x;
    unsigned long long out;
    if (j < 6) {
      double sum = 0.;
      for (int w = 0; w < n_warps; ++w) sum += __longlong_as_double((long long)s_part[w][j]);
      out = (unsigned long long)__double_as_longlong(sum);
    } else if (j == 6) {
      out = 0ull;
      for (int w = 0; w < n_warps; ++w) out += s_part[w][6];
    } else {
      out = ((unsigned long long)(b + 1) << kTagShift) | ((unsigned long long)x0 << kX0Shift) |
            ((unsigned long long)m0bits << kM0Shift);       // sample tag and the shift of the sums
      for (int w = 0; w < n_warps; ++w) out |= s_part[w][7];
    }
    slot[j] = out;
  }
}

// Rows of x that start on any 2-byte boundary (the compressed-signal layout with a row width that
// is a multiple of 8): a lane's 8 elements straddle two aligned 16-byte words.  The misalignment
// `s` (bytes, even) is the same for every chunk of a row.  A lane loads the aligned word below its
// chunk; the word above it is its neighbour's, fetched by a shuffle -- or by a load of its own
// for lane 31 and for the last chunk of the row, where no neighbour holds it -- and a funnel
// shift by s puts the 8 elements in place.  Past the end of the tensor (last chunk of the last row)
// the upper word is put together from 2-byte loads of the elements that exist.
__device__ __forceinline__ uint4 shifted_chunk(const uint4 &w0, const uint4 &w1, unsigned s) {
  const unsigned in[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
  const unsigned bs = (s & 3u) * 8u;
  uint4 out;
  switch (s >> 2) {                     // the same for the whole warp
    case 0:
      out.x = __funnelshift_r(in[0], in[1], bs); out.y = __funnelshift_r(in[1], in[2], bs);
      out.z = __funnelshift_r(in[2], in[3], bs); out.w = __funnelshift_r(in[3], in[4], bs);
      break;
    case 1:
      out.x = __funnelshift_r(in[1], in[2], bs); out.y = __funnelshift_r(in[2], in[3], bs);
      out.z = __funnelshift_r(in[3], in[4], bs); out.w = __funnelshift_r(in[4], in[5], bs);
      break;
    case 2:
      out.x = __funnelshift_r(in[2], in[3], bs); out.y = __funnelshift_r(in[3], in[4], bs);
      out.z = __funnelshift_r(in[4], in[5], bs); out.w = __funnelshift_r(in[5], in[6], bs);
      break;
    default:
      out.x = __funnelshift_r(in[3], in[4], bs); out.y = __funnelshift_r(in[4], in[5], bs);
      out.z = __funnelshift_r(in[5], in[6], bs); out.w = __funnelshift_r(in[6], in[7], bs);
      break;
  }
  return out;
}

// (row_first, x_extent: where the row starts in x and how many elements x has, for the checked
// build: an aligned word may begin up to 7 elements below the row and end as many above it, inside
// the 16-byte granule the row's first or last element lies in -- except past the last row, which
// is why that row's upper word is put together from the elements that exist)
template <int kU>
__device__ __forceinline__ void load_x_shifted(const uint16_t *row_ptr, int base, int chunks, bool last_row,
                                               const bool (&ok)[kU], uint4 (&xv)[kU], long long row_first,
                                               long long x_extent) {
  const int lane = threadIdx.x & 31;
  const unsigned s = (unsigned)(reinterpret_cast<uintptr_t>(row_ptr) & 15u);
  if (s == 0u) {
#pragma unroll
    for (int u = 0; u < kU; ++u)
      if (ok[u] && SENTINEL_BOUNDS(kSiteX, row_first + (long long)(base + u * 32 + lane) * 8, 8, x_extent))
        xv[u] = ld_x128(row_ptr + (size_t)(base + u * 32 + lane) * 8);
    return;
  }
  const uint16_t *al = row_ptr - (s >> 1);                 // 16-byte aligned
  // all loads first (the few lanes that fetch their own upper word included), then the shuffles
  uint4 w0[kU], own[kU];
  bool direct[kU];
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    const int c = base + u * 32 + lane;
    w0[u] = own[u] = make_uint4(0u, 0u, 0u, 0u);
    direct[u] = ok[u] && (lane == 31 || c + 1 >= chunks);  // nobody holds the word above this chunk
    // (in elements of x: the aligned word below chunk c begins at row_first - s/2 + 8c)
    [[maybe_unused]] const long long lower = row_first - (long long)(s >> 1) + (long long)c * 8;
    if (ok[u] && SENTINEL_BOUNDS(kSiteX, lower + 7, 1, x_extent + 7)) w0[u] = ld_x128(al + (size_t)c * 8);
    if (direct[u]) {
      const uint16_t *up = al + (size_t)(c + 1) * 8;
      if (last_row && c + 1 >= chunks) {                   // only its first s bytes exist for sure
        unsigned e[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (SENTINEL_BOUNDS(kSiteX, lower + 8, (long long)(s >> 1), x_extent))
          for (unsigned k = 0; k < (s >> 1); ++k) e[k] = up[k];
        own[u] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
      } else if (SENTINEL_BOUNDS(kSiteX, lower + 8, 1, x_extent)) {   // (the word above a row that is not the last begins inside x)
        own[u] = ld_x128(up);
      }
    }
  }
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    uint4 w1;
    w1.x = __shfl_down_sync(0xffffffffu, w0[u].x, 1);
    w1.y = __shfl_down_sync(0xffffffffu, w0[u].y, 1);
    w1.z = __shfl_down_sync(0xffffffffu, w0[u].z, 1);
    w1.w = __shfl_down_sync(0xffffffffu, w0[u].w, 1);
    if (direct[u]) w1 = own[u];
    if (ok[u]) xv[u] = shifted_chunk(w0[u], w1, s);
  }
}

// ---------------------------------------------------------------------------------------------
// streaming phase
//
// Streaming CTA c owns the rows [c*R/G, (c+1)*R/G) of the flat [B*T, d] view (R = B*T rows, G
// streaming CTAs), so every CTA moves the same number of bytes to within one row.  Inside the
// CTA the rows are cut into warp tiles of 32*kUnroll chunks (512 elements) that never cross a
// row, dealt round-robin to the warps, so the warps finish within one tile of each other.  A
// CTA's rows can straddle one sample boundary (the host guarantees at most one), hence two
// partial slots per CTA, each tagged with its sample.

constexpr int kSegsPerCta = 2;

// kScalar: the layout of a subspace-compressed signal, x[:, :, :-1] of a [B,T,k+1] tensor (SWARM
// appendix): rows of x are row_stride elements apart and start on any 2-byte boundary, and d
// need not be a multiple of 8.  Lanes then own interleaved columns (col = tile + q*32 + lane),
// so that every 2-byte / 4-byte access of a warp is contiguous; the arithmetic is the same.
template <bool kScalar, bool kBf16, bool kShifted>
__device__ void stream_segment(const StreamArgs &a, int b, long long ra, long long rb,
                               const void *m_in, void *m_out,
                               unsigned long long (*s_part)[kSlotWords],
                               unsigned long long *slot) {
  // chunks per lane and trip: with a bf16 reference a chunk brings 32 bytes instead of 48, so
  // a trip takes more of them to keep as many bytes in flight
  constexpr int kU = (kBf16 && !kScalar) ? kUnrollBf16 : kUnroll;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = (a.d + 7) >> 3;
  const int tiles_per_row = (chunks + 32 * kU - 1) / (32 * kU);
  const int n_tiles = (int)(rb - ra) * tiles_per_row;       // < 2^31: rows/G * d/1024
  const size_t sample_off = (size_t)b * a.T * a.d;
  const bool write_ema = (m_out != nullptr);
  const bool tokens = (a.token_out != nullptr);
  const float beta = a.beta, omb = a.one_minus_beta;

  const unsigned x0 = SENTINEL_BOUNDS(kSiteX, (long long)b * a.T * a.x_row_stride, 1, a.x_extent)
                          ? a.x[(size_t)b * a.T * (size_t)a.x_row_stride] : 0u;
  const unsigned x0pair = x0 | (x0 << 16);
  const unsigned m0bits = SENTINEL_BOUNDS(kSiteRefIn, sample_off, 1, a.ref_extent)
                              ? __float_as_uint(load_m1<kBf16>(m_in, sample_off)) : 0u;

  ThreadAcc t = {0., 0., 0., 0., 0., 0., 0u, 0u, 0u, 0u};

  // tile j = (row rr, segment seg); j advances by kWarps, so (rr, seg) advance by a fixed step
  const int step_rr = kWarps / tiles_per_row, step_seg = kWarps % tiles_per_row;
  int rr = warp / tiles_per_row, seg = warp % tiles_per_row;
  for (int j = warp; j < n_tiles; j += kWarps) {
    const long long row = ra + rr;
    const size_t off = (size_t)row * a.d;
    const int base = seg * 32 * kU;
    GroupAcc g = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0u};

    if (kScalar) {
      constexpr int kPerLane = 8 * kUnroll;
      const size_t off_x = (size_t)row * (size_t)a.x_row_stride;
      const int col0 = base * 8 + lane;
      const float x0f = __uint_as_float(x0 << 16), m0f = __uint_as_float(m0bits);
      unsigned short xs[kPerLane];
      float ms[kPerLane];
#pragma unroll
      for (int q = 0; q < kPerLane; ++q) {
        const int col = col0 + q * 32;
        if (col < a.d && SENTINEL_BOUNDS(kSiteX, off_x + col, 1, a.x_extent) &&
            SENTINEL_BOUNDS(kSiteRefIn, off + col, 1, a.ref_extent)) {
          xs[q] = a.x[off_x + col];
          ms[q] = load_m1<kBf16>(m_in, off + col);
        }
      }
#pragma unroll
      for (int q = 0; q < kPerLane; ++q) {
        const int col = col0 + q * 32;
        if (col < a.d) {
          const unsigned xb = xs[q];
          t.nf_bits |= ((xb & 0x7F80u) == 0x7F80u) ? 1u : 0u;
          t.x_diff |= xb ^ x0;
          t.m_diff |= __float_as_uint(ms[q]) ^ m0bits;
          const float xf = __uint_as_float(xb << 16);
          element(xf, ms[q], x0f, m0f, g);
          if (write_ema && SENTINEL_BOUNDS(kSiteRefOut, off + col, 1, a.ref_extent))
            store_m1<kBf16>(m_out, off + col, fmaf(beta, ms[q], omb * xf));
        }
      }
    } else {
      uint4 xv[kU];
      F8 mv[kBf16 ? 1 : kU];
      uint4 mraw[kBf16 ? kU : 1];          // a bf16 reference stays packed until its chunk is worked on
      bool ok[kU];
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int c = base + u * 32 + lane;
        ok[u] = c < chunks && SENTINEL_BOUNDS(kSiteRefIn, off + (size_t)c * 8, 8, a.ref_extent) &&
                (kShifted || SENTINEL_BOUNDS(kSiteX, off + (size_t)c * 8, 8, a.x_extent));
        if (ok[u]) {
          if (!kShifted) xv[u] = ld_x128(a.x + off + (size_t)c * 8);
          if (kBf16) mraw[u] = ld_x128(static_cast<const uint16_t *>(m_in) + off + (size_t)c * 8);
          else mv[u] = ld_m256(static_cast<const float *>(m_in) + off + (size_t)c * 8);
        }
      }
      if (kShifted)
        load_x_shifted<kU>(a.x + (size_t)row * (size_t)a.x_row_stride, base, chunks,
                           row == (long long)a.B * a.T - 1, ok, xv, row * a.x_row_stride, a.x_extent);
      if (kBf16) {
        // the packed path (see chunk_packed): m0 is a bf16 value here, m0bits >> 16 its pattern
        PairAcc p = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, 0u, 0x7F7F7F7Fu};
        const unsigned m0pair = (m0bits >> 16) | (m0bits & 0xFFFF0000u);
        const float x0f = __uint_as_float(x0 << 16), m0f = __uint_as_float(m0bits);
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          if (ok[u]) {
            uint4 cand;
            chunk_packed(xv[u], mraw[u], cand, p, t, x0pair, m0pair, x0f, m0f, beta, omb, write_ema);
            if (write_ema)
              asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};"
                           :: "l"(static_cast<uint16_t *>(m_out) + off + (size_t)(base + u * 32 + lane) * 8),
                              "r"(cand.x), "r"(cand.y), "r"(cand.z), "r"(cand.w) : "memory");
          }
        }
        unsigned flips = p.flips / kFlipUnit;
        // an exact zero in x or m somewhere in this trip: count again, element by element
        if (__any_sync(0xffffffffu, ((p.zmin & 0x7FFFu) == 0u) || ((p.zmin & 0x7FFF0000u) == 0u))) {
          flips = 0u;
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if (ok[u]) flips += flips_exact(xv[u], mraw[u]);
        }
        const float ab = p.ab[0] + p.ab[1];
        if (__any_sync(0xffffffffu, !(ab <= 3.4028234664e38f))) {   // not a finite sum: look at the bits
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if (ok[u]) t.nf_bits |= nonfinite_bits(xv[u]);
        }
        g.sx = p.sx.lo + p.sx.hi;     g.sxx = p.sxx.lo + p.sxx.hi;
        g.sm = p.sm.lo + p.sm.hi;     g.smm = p.smm.lo + p.smm.hi;
        g.sxm = p.sxm.lo + p.sxm.hi;  g.ab = ab;
        g.flips = flips;
      } else {
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          if (ok[u]) {
            chunk(xv[u], mv[u], g, t, x0pair, m0bits, beta, omb, write_ema);
            if (write_ema) store_m8<kBf16>(m_out, off + (size_t)(base + u * 32 + lane) * 8, mv[u]);
          }
        }
      }
    }
    // fold the short fp32 run into the fp64 accumulators
    t.sx += (double)g.sx;   t.sxx += (double)g.sxx;
    t.sm += (double)g.sm;   t.smm += (double)g.smm;
    t.sxm += (double)g.sxm; t.ab += (double)g.ab;
    t.flips += g.flips;

    if (tokens) {                       // this tile's share of the token's sums
      const float sx = warp_sum(g.sx), sxx = warp_sum(g.sxx), ab = warp_sum(g.ab);
      const float fl = warp_sum((float)g.flips);
      if (lane == 0 && SENTINEL_BOUNDS(kSiteToken, row, 1, (long long)a.B * a.T) &&
          SENTINEL_BOUNDS(kSiteToken, seg, 1, tiles_per_row)) {
        float4 *dst = (tiles_per_row == 1) ? reinterpret_cast<float4 *>(a.token_out) + row
                                           : reinterpret_cast<float4 *>(a.token_part) + row * tiles_per_row + seg;
        float4 v = make_float4(sx, sxx, ab, fl);
        if (tiles_per_row == 1) {       // back from shifted to raw sums over the d channels
          const float x0f = __uint_as_float(x0 << 16), dd = (float)a.d;
          v.y = fmaf(dd * x0f, x0f, fmaf(2.f * x0f, sx, sxx));
          v.x = fmaf(dd, x0f, sx);
        }
        *dst = v;
      }
    }
    rr += step_rr;
    seg += step_seg;
    if (seg >= tiles_per_row) { seg -= tiles_per_row; ++rr; }
  }

  if (tokens && tiles_per_row > 1) {    // a row's tiles went to several warps: add them in order
    __syncthreads();
    const float x0f = __uint_as_float(x0 << 16), dd = (float)a.d;
    for (long long row = ra + threadIdx.x; row < rb; row += kThreads) {
      const float4 *src = reinterpret_cast<const float4 *>(a.token_part) + row * tiles_per_row;
      float4 acc = __ldcg(src);
      for (int sgm = 1; sgm < tiles_per_row; ++sgm) {
        const float4 v = __ldcg(src + sgm);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      const float raw_sx = fmaf(dd, x0f, acc.x);
      const float raw_sxx = fmaf(dd * x0f, x0f, fmaf(2.f * x0f, acc.x, acc.y));
      reinterpret_cast<float4 *>(a.token_out)[row] = make_float4(raw_sx, raw_sxx, acc.z, acc.w);
    }
  }

  reduce_to_slot(t, b, x0, m0bits, s_part, slot);
}

template <bool kScalar, bool kBf16, bool kShifted>
__device__ void stream_cta(const StreamArgs &a, int c, const void *m_in, void *m_out,
                           unsigned long long (*s_part)[kSlotWords]) {
  const long long R = (long long)a.B * a.T;
  const long long R0 = (R * c) / a.G, R1 = (R * (c + 1)) / a.G;
  long long ra = R0;
  for (int sgm = 0; sgm < kSegsPerCta; ++sgm) {
    unsigned long long *slot = a.partials + ((size_t)c * kSegsPerCta + sgm) * kSlotWords;
    if (!SENTINEL_BOUNDS(kSiteSlot, ((size_t)c * kSegsPerCta + sgm) * kSlotWords, kSlotWords, a.partials_words)) continue;
    if (ra < R1) {
      const int b = (int)(ra / a.T);
      const long long sample_end = (long long)(b + 1) * a.T;
      const long long rb = sample_end < R1 ? sample_end : R1;
      stream_segment<kScalar, kBf16, kShifted>(a, b, ra, rb, m_in, m_out, s_part, slot);
      ra = rb;
    } else if (threadIdx.x == 0) {
      slot[7] = 0ull;                   // tag 0: unused
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Alg. 5 on the device (one CTA)

__device__ __forceinline__ double percentile_sorted(const double *s, int n, double p) {
  const double pos = __dmul_rn(p, (double)(n - 1));
  const int lo = (int)floor(pos);
  const int hi = (lo + 1 < n) ? lo + 1 : lo;
  const double frac = __dsub_rn(pos, (double)lo);
  return __dadd_rn(s[lo], __dmul_rn(frac, __dsub_rn(s[hi], s[lo])));
}

// History layout.  A window of at most `cap` entries lives in a ring of cap + units slots
// (units = entries one step can append: 1 at level 0, B at level 1), so the entries a step
// pushes out stay readable until the next step appends: the refresh that follows a step finds
// both what joined and what left.  Next to each ring the same window is kept in ascending
// order; a refresh merges the few changes into it instead of sorting the window again.
__host__ __device__ inline int ring_size(int cap, int units) { return cap + units; }
__host__ __device__ inline size_t ring_offset(int L, int i, int cap0, int cap1, int units0, int units1) {
  return L ? (size_t)kNumMetrics * ring_size(cap0, units0) + (size_t)i * ring_size(cap1, units1)
           : (size_t)i * ring_size(cap0, units0);
}
__host__ __device__ inline size_t sorted_offset(int L, int i, int cap0, int cap1) {
  return L ? (size_t)kNumMetrics * cap0 + (size_t)i * cap1 : (size_t)i * cap0;
}

// One thread group per (level, metric) window: three warps each with three metrics in use, two
// with four.
__host__ __device__ inline int refresh_group_threads(int n_metrics, int cta_threads) {
  return (cta_threads / (2 * n_metrics)) & ~31;
}
constexpr int kMinThreads = 2 * kNumMetrics * 64;   // one thread group of two warps per window at least
static_assert(kMinThreads <= kThreads, "one thread group per window");

__device__ __forceinline__ void group_barrier(int group, int group_threads) {   // named barrier 1 + group
  asm volatile("bar.sync %0, %1;" :: "r"(group + 1), "r"(group_threads) : "memory");
}

// doubles of shared memory the refresh needs: per window the old and the new ascending copy
// (cap each), a staging area for what left and what joined (2*units) and their sorted lists
// (units each)
__host__ __device__ inline size_t window_smem_doubles(int cap, int units) {
  return 2 * (size_t)cap + 4 * (size_t)units;
}
__host__ __device__ inline size_t refresh_smem_doubles(int cap0, int cap1, int units0, int units1, int n_metrics) {
  return (size_t)n_metrics * (window_smem_doubles(cap0, units0) + window_smem_doubles(cap1, units1));
}

__device__ __forceinline__ int lower_bound(const double *a, int n, double v) {   // # entries < v
  int lo = 0, hi = n;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] < v) lo = mid + 1; else hi = mid; }
  return lo;
}
__device__ __forceinline__ int upper_bound(const double *a, int n, double v) {   // # entries <= v
  int lo = 0, hi = n;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] <= v) lo = mid + 1; else hi = mid; }
  return lo;
}

// # entries of the ascending array s that are < x (strict) or <= x, found by one warp in two
// rounds: 32 evenly spaced probes pick a block, then the block is scanned
template <bool kOrEqual>
__device__ __forceinline__ int warp_rank(const double *s, int n, double x, int lane) {
  const int stride = (n + 31) >> 5;
  const int i0 = lane * stride;
  const bool below0 = (i0 < n) && (kOrEqual ? (s[i0] <= x) : (s[i0] < x));
  const int c = __popc(__ballot_sync(0xffffffffu, below0));   // block starts below x: a prefix
  if (c == 0) return 0;
  const int base = (c - 1) * stride;
  int count = base;
  for (int t = 0; t < stride; t += 32) {
    const int idx = base + t + lane;
    const bool below = (t + lane < stride) && (idx < n) && (kOrEqual ? (s[idx] <= x) : (s[idx] < x));
    count += __popc(__ballot_sync(0xffffffffu, below));
  }
  return count;
}

// entries strictly outside [lo, hi] of an ascending window
__device__ __forceinline__ int warp_count_outside(const double *s, int n, double lo, double hi, int lane) {
  return warp_rank<false>(s, n, lo, lane) + (n - warp_rank<true>(s, n, hi, lane));
}

// Refreshes q1,q2,q3,k,tau of every (level, metric) window of one kind (Alg. 5).  Whole CTA:
// the windows are handled side by side, each by a group of warps with its own named barrier.
__device__ void refresh_thresholds(KindState *ks, const double *hist, double *sorted, int cap0, int cap1,
                                   int units0, int units1, int n_metrics, const Alg5Params &a5, double *s_dyn) {
  const int group_threads = refresh_group_threads(n_metrics, (int)blockDim.x);   // any CTA of kMinThreads or more
  const int group = threadIdx.x / group_threads;
  const int gt = threadIdx.x - group * group_threads;
  if (group < 2 * n_metrics) {
    const int L = group / n_metrics, i = group - L * n_metrics;
    const int n = ks->hist_count[L];
    if (n > 0) {                                   // an empty window leaves everything as it is
      const int cap = L ? cap1 : cap0, units = L ? units1 : units0, size = ring_size(cap, units);
      const int joined = ks->last_joined[L], evicted = ks->last_evicted[L], head = ks->hist_head[L];
      const int n_old = n - joined + evicted;
      const double *ring = hist + ring_offset(L, i, cap0, cap1, units0, units1);
      double *srt = sorted + sorted_offset(L, i, cap0, cap1);
      // this window's shared memory: old copy, new copy, staging, what left, what joined
      double *s_old = s_dyn + (L ? (size_t)n_metrics * window_smem_doubles(cap0, units0) +
                                       (size_t)i * window_smem_doubles(cap1, units1)
                                 : (size_t)i * window_smem_doubles(cap0, units0));
      double *s_new = s_old + cap, *s_stage = s_new + cap, *s_out = s_stage + 2 * units, *s_in = s_out + units;

#ifdef SENTINEL_CHECK_BOUNDS
      const bool window_ok = SENTINEL_BOUNDS(kSiteSorted, n_old, 0, cap) && SENTINEL_BOUNDS(kSiteSorted, n, 0, cap) &&
                             SENTINEL_BOUNDS(kSiteRing, evicted, 0, units) && SENTINEL_BOUNDS(kSiteRing, joined, 0, units) &&
                             SENTINEL_BOUNDS(kSiteRing, head, 1, size);
      if (!window_ok) { group_barrier(group, group_threads); group_barrier(group, group_threads); group_barrier(group, group_threads); }
      if (window_ok) {
#endif
      for (int p = gt; p < n_old; p += group_threads) s_old[p] = srt[p];
      // the entries pushed out sit just before the head, the ones that joined at the tail;
      // stage them, then rank-sort them (they are few) into s_out / s_in
      for (int j = gt; j < evicted; j += group_threads) s_stage[j] = ring[(head - evicted + j + size) % size];
      for (int j = gt; j < joined; j += group_threads) s_stage[evicted + j] = ring[(head + n - joined + j) % size];
      group_barrier(group, group_threads);
      for (int j = gt; j < evicted + joined; j += group_threads) {
        const bool is_out = j < evicted;
        const double *src = is_out ? s_stage : s_stage + evicted;
        const int m = is_out ? evicted : joined, jj = is_out ? j : j - evicted;
        const double v = src[jj];
        int rank = 0;
        for (int q = 0; q < m; ++q) rank += (src[q] < v) || (src[q] == v && q < jj);
        (is_out ? s_out : s_in)[rank] = v;
      }
      group_barrier(group, group_threads);
      // merge: old entries keep their order, lose the first copies of what left, and make
      // room for what joined (a joining value goes after equal old ones)
      for (int p = gt; p < n_old; p += group_threads) {
        const double v = s_old[p];
        const int out_lt = lower_bound(s_out, evicted, v);
        const int out_eq = upper_bound(s_out, evicted, v) - out_lt;
        int gone_before = out_lt;
        bool gone = false;
        if (out_eq > 0) {                          // v is a value that left: its first copies go
          const int copy = p - lower_bound(s_old, n_old, v);
          gone = copy < out_eq;
          gone_before += gone ? copy : out_eq;
        }
        if (!gone) s_new[p - gone_before + lower_bound(s_in, joined, v)] = v;
      }
      for (int j = gt; j < joined; j += group_threads) {
        const double v = s_in[j];
        s_new[j + upper_bound(s_old, n_old, v) - upper_bound(s_out, evicted, v)] = v;
      }
      group_barrier(group, group_threads);
      for (int p = gt; p < n; p += group_threads) srt[p] = s_new[p];

      if (gt < 32) {                               // the group's first warp walks the steps
        const int lane = gt;
        const double *s_sort = s_new;
        const double q1 = percentile_sorted(s_sort, n, 0.25);
        const double q2 = percentile_sorted(s_sort, n, 0.50);
        const double q3 = percentile_sorted(s_sort, n, 0.75);
        const double iqr = fmax(__dsub_rn(q3, q1), a5.eps);
        const double dn = (double)n;
        // FP-rate = count/n is monotone in the count, so "FP-rate > alpha" and
        // "FP-rate < shrink_ratio*alpha" are thresholds on the count, found once with the
        // very division the comparison is defined by
        const double low_mark = __dmul_rn(a5.shrink_ratio, a5.alpha);
        int widen_from = (int)floor(a5.alpha * dn) - 1;       // smallest count with count/n > alpha
        if (widen_from < 0) widen_from = 0;
        while (widen_from <= n && !((double)widen_from / dn > a5.alpha)) ++widen_from;
        int narrow_to = (int)ceil(low_mark * dn) + 1;         // largest count with count/n < low_mark
        if (narrow_to > n) narrow_to = n;
        while (narrow_to >= 0 && !((double)narrow_to / dn < low_mark)) --narrow_to;

        double k = ks->thr[L][i][3];
        double lo = __dsub_rn(q2, __dmul_rn(k, iqr));
        double hi = __dadd_rn(q2, __dmul_rn(k, iqr));
        int outside = warp_count_outside(s_sort, n, lo, hi, lane);
        int it = 0;
        while (outside >= widen_from && it < a5.n_max) {      // widen
          k = __dmul_rn(k, a5.gamma_g);
          lo = __dsub_rn(q2, __dmul_rn(k, iqr));
          hi = __dadd_rn(q2, __dmul_rn(k, iqr));
          outside = warp_count_outside(s_sort, n, lo, hi, lane);
          ++it;
        }
        it = 0;
        while (outside <= narrow_to && it < a5.n_max) {       // narrow
          k = __dmul_rn(k, a5.gamma_s);
          lo = __dsub_rn(q2, __dmul_rn(k, iqr));
          hi = __dadd_rn(q2, __dmul_rn(k, iqr));
          outside = warp_count_outside(s_sort, n, lo, hi, lane);
          ++it;
        }
        const double d_min = __dmul_rn(fabs(q2), a5.lambda);
        lo = fmin(lo, __dsub_rn(q2, d_min));
        hi = fmax(hi, __dadd_rn(q2, d_min));
        if (lane == 0) {
          double *t = ks->thr[L][i];
          t[0] = q1; t[1] = q2; t[2] = q3; t[3] = k; t[4] = lo; t[5] = hi;
          ks->has_thr[L][i] = 1;
        }
      }
#ifdef SENTINEL_CHECK_BOUNDS
      }
#endif
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    ks->refresh_pending = 0;
    ks->last_joined[0] = ks->last_joined[1] = 0;   // the sorted copies are up to date
    ks->last_evicted[0] = ks->last_evicted[1] = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// finalize: last CTA only

struct UnitSums {
  double s[6];               // sums of (x-x0) (x-x0)^2 (m-m0) (m-m0)^2 (x-x0)(m-m0) |x-m|
  unsigned long long flips;
  unsigned long long bits;
  unsigned long long first;  // bits 0-15 first x (bf16), bits 16-47 first m (fp32)
  double x0, m0;             // the shift the sums were taken about
};

// What one pass of finalize reports on: a single submission, or one worker of an iteration.
struct FinalizeTarget {
  int worker;                            // whose counters move (0 for a single submission)
  const unsigned long long *partials;    // that tensor's partial slots
  float *scores_out;                     // [(1+B)*n_metrics] or nullptr
  unsigned *flags_out;                   // [1+B] or nullptr
  const float *sw;                       // [1+B] sliced Wasserstein distances, or nullptr
  int elsewhere;                         // the worker was tainted at another stage: not collected
  int last;                              // the launch ends with this pass: the ticket is re-armed
  int per_sample_blocks;                 // slots laid out [sample][CTA][segment] (every CTA has rows of every
                                         // sample) instead of [CTA][segment] tagged with the sample
};

__device__ void finalize(const StreamArgs &a, const FinalizeTarget &ft) {
  __shared__ UnitSums s_unit[kMaxB + 1];
  __shared__ unsigned s_flag[kMaxB + 1];
  __shared__ int s_severe, s_no_thr;
  __shared__ unsigned s_status;                  // status bits of row 0
  // The handle's small state is fetched once, in one batch, and written back once: by now it
  // has long left the L2, and touching it field by field would cost a DRAM round trip each.
  __shared__ __align__(8) HandleState s_hs;
  static_assert(sizeof(HandleState) % 8 == 0, "copied as 64-bit words");
  constexpr int kStateWords = (int)(sizeof(HandleState) / 8);
  static_assert(kStateWords <= kMinThreads, "one thread per word of the state");
  const int n_threads = (int)blockDim.x, n_warps = n_threads >> 5;   // (kernels of several CTA sizes end here)
  const int kDecider = n_threads - 1;            // the thread that keeps the counters

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int B = a.B, rows = B + 1;
  const size_t Ns = (size_t)a.T * a.d;

  if (tid == 0) { s_severe = 0; s_no_thr = 0; s_status = 0u; }
  if (a.hs && tid >= n_threads - kStateWords) {     // the last warps: the first ones gather sums
    const int w = tid - (n_threads - kStateWords);
    reinterpret_cast<unsigned long long *>(&s_hs)[w] =
        __ldcg(reinterpret_cast<const unsigned long long *>(a.hs) + w);
  }

  // per-sample sums over the slots tagged with that sample, in CTA order
  for (int b = warp; b < B; b += n_warps) {
    double v[6] = {0., 0., 0., 0., 0., 0.};
    unsigned long long fl = 0ull, bits = 0ull, first = 0ull;
    // streaming CTAs whose rows can touch sample b (a superset; the tag decides)
    const long long R = (long long)B * a.T;
    long long c_lo = ((long long)b * a.T * a.G) / R - 1, c_hi = ((long long)(b + 1) * a.T * a.G + R - 1) / R;
    if (c_lo < 0) c_lo = 0;
    if (c_hi > a.G - 1) c_hi = a.G - 1;
    const unsigned long long *block = ft.partials;
    if (ft.per_sample_blocks) {              // sample b's own block: a slot pair from every CTA
      c_lo = 0;
      c_hi = a.G - 1;
      block += (size_t)b * a.G * kSegsPerCta * kSlotWords;
    }
    const long long n_slots = (c_hi - c_lo + 1) * kSegsPerCta;
    for (long long q = lane; q < n_slots; q += 32) {
      const unsigned long long *slot = block + ((size_t)c_lo * kSegsPerCta + q) * kSlotWords;
      if (!SENTINEL_BOUNDS(kSiteSlot, c_lo * kSegsPerCta + q, 1, (long long)a.G * kSegsPerCta)) continue;
      unsigned long long w[kSlotWords];
#pragma unroll
      for (int j = 0; j < kSlotWords; ++j) w[j] = __ldcg(slot + j);   // one round trip, then the tag
      const unsigned long long tag = (w[7] >> kTagShift) & 0xFFull;
      if (ft.per_sample_blocks ? (tag == 0ull) : (tag != (unsigned long long)(b + 1))) continue;
#pragma unroll
      for (int j = 0; j < 6; ++j) v[j] += __longlong_as_double((long long)w[j]);
      fl += w[6];
      bits |= w[7] & 0x7ull;
      first = w[7] >> kX0Shift;          // the same in every slot of this sample
    }
#pragma unroll
    for (int j = 0; j < 6; ++j) v[j] = warp_sum(v[j]);
    fl = warp_sum(fl);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      bits |= __shfl_xor_sync(0xffffffffu, bits, o);
      first |= __shfl_xor_sync(0xffffffffu, first, o);
    }
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < 6; ++j) s_unit[1 + b].s[j] = v[j];
      s_unit[1 + b].flips = fl;
      s_unit[1 + b].bits = bits;
      s_unit[1 + b].first = first;
      s_unit[1 + b].x0 = (double)__uint_as_float(((unsigned)first & 0xFFFFu) << 16);
      s_unit[1 + b].m0 = (double)__uint_as_float((unsigned)(first >> 16));
    }
  }
  __syncthreads();

  // whole-tensor unit = the samples added up (warp 0, fixed tree), re-centred on sample 0's
  // shift K: sum (x-K) = sum (x-x0) + n dx,  sum (x-K)^2 = sum (x-x0)^2 + 2 dx sum (x-x0) + n dx^2,
  // sum (x-Kx)(m-Km) = sum (x-x0)(m-m0) + dx sum (m-m0) + dm sum (x-x0) + n dx dm
  if (warp == 0) {
    const UnitSums &ref = s_unit[1];
    const double n = (double)Ns;
    double t[6] = {0., 0., 0., 0., 0., 0.};
    unsigned long long fl = 0ull, bits = 0ull;
    for (int b = lane; b < B; b += 32) {
      const UnitSums &v = s_unit[1 + b];
      const double dx = v.x0 - ref.x0, dm = v.m0 - ref.m0;
      t[0] += v.s[0] + n * dx;
      t[1] += v.s[1] + 2. * dx * v.s[0] + n * dx * dx;
      t[2] += v.s[2] + n * dm;
      t[3] += v.s[3] + 2. * dm * v.s[2] + n * dm * dm;
      t[4] += v.s[4] + dx * v.s[2] + dm * v.s[0] + n * dx * dm;
      t[5] += v.s[5];
      fl += v.flips;
      bits |= v.bits;
      if ((v.first & 0xFFFFull) != (ref.first & 0xFFFFull)) bits |= kBitXVaries;
      if ((v.first >> 16) != (ref.first >> 16)) bits |= kBitMVaries;
    }
#pragma unroll
    for (int j = 0; j < 6; ++j) t[j] = warp_sum(t[j]);
    fl = warp_sum(fl);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < 6; ++j) s_unit[0].s[j] = t[j];
      s_unit[0].flips = fl;
      s_unit[0].bits = bits;
      s_unit[0].first = ref.first;
      s_unit[0].x0 = ref.x0;
      s_unit[0].m0 = ref.m0;
    }
  }
  __syncthreads();

  KindState *ks = a.hs ? &s_hs.kind[a.kind] : nullptr;     // the shared copy
  const bool replica = (a.mode == kModeReplicaVerify || a.mode == kModeReplicaWarmup);
  const bool testing = (a.mode == kModeVerify || a.mode == kModeReplicaVerify);
  const int w = replica ? ft.worker : 0;                     // whose counters this pass moves

  // banned, or tainted at another stage (Alg. 3; left out of the loop of Alg. 2): not
  // collected, only reported
  if (a.mode == kModeReplicaVerify && (s_hs.banned[w] || ft.elsewhere)) {
    const bool banned = s_hs.banned[w] != 0;
    if (tid < rows) {
      if (ft.scores_out)
        for (int i = 0; i < a.n_metrics; ++i) ft.scores_out[tid * a.n_metrics + i] = CUDART_NAN_F;
      if (ft.flags_out) ft.flags_out[tid] = tid == 0 ? (banned ? kFlagBanned : kFlagTaintedElsewhere) : 0u;
    }
    if (tid == kDecider) {
      if (w == 0) {                                          // the iteration still starts here
        ks->steps += 1;
        ks->step_collected = ks->step_tainted = ks->step_nonfinite = ks->step_elsewhere = 0u;
      }
      if (!banned) ks->step_elsewhere |= 1u << w;
      ks->refresh_pending = 1;                               // Alg. 5 still runs once per iteration
      if (ft.last) s_hs.ticket = 0u;
    }
    __syncthreads();
    if (tid < kStateWords)
      reinterpret_cast<unsigned long long *>(a.hs)[tid] = reinterpret_cast<unsigned long long *>(&s_hs)[tid];
    return;
  }

  // scores and the Tukey test: one thread per unit
  unsigned my_flag = 0u;
  double g[kNumMetrics] = {0., 0., 0., 0.};
  double st_var_x = 0., st_var_m = 0., st_cov = 0., st_rho = 0., inv_n = 0.;
  bool nonfinite = false;
  int ring_head = 0, ring_count = 0;              // this unit's level, before this step
  if (tid < rows) {
    const UnitSums &u = s_unit[tid];
    const double n = (tid == 0) ? (double)B * (double)Ns : (double)Ns;
    inv_n = 1. / n;
    nonfinite = (u.bits & kBitNonfinite) != 0ull;
    // a vector whose elements all equal its first one (bitwise, or +0 against -0) has
    // variance exactly 0
    const bool x_const = !(u.bits & kBitXVaries) || u.s[1] == 0.;
    const bool m_const = !(u.bits & kBitMVaries) || u.s[3] == 0.;
    const double dmean_x = u.s[0] * inv_n, dmean_m = u.s[2] * inv_n;   // means of the shifted values
    st_var_x = x_const ? 0. : fmax(u.s[1] * inv_n - dmean_x * dmean_x, 0.);
    st_var_m = m_const ? 0. : fmax(u.s[3] * inv_n - dmean_m * dmean_m, 0.);
    st_cov = u.s[4] * inv_n - dmean_x * dmean_m;
    double l2z;
    if (st_var_x > 0. && st_var_m > 0.) {
      st_rho = fmin(fmax(st_cov * rsqrt(st_var_x) * rsqrt(st_var_m), -1.), 1.);
      l2z = 2. - 2. * st_rho;                 // mean (zx - zm)^2 = 2 - 2 rho
    } else {
      l2z = (st_var_x > 0. || st_var_m > 0.) ? 1. : 0.;   // a constant vector z-scores to zero
    }
    g[0] = u.s[5] * inv_n;
    g[1] = l2z;
    g[2] = (double)u.flips * inv_n;
    if (ft.sw) g[3] = (double)__ldcg(ft.sw + tid);   // left by the launches that precede this one
    if (nonfinite) {
      for (int i = 0; i < kNumMetrics; ++i) g[i] = CUDART_NAN;
      my_flag = kFlagNonfinite;
    } else if (testing) {
      const int L = (tid == 0) ? 0 : 1;
#pragma unroll
      for (int i = 0; i < kNumMetrics; ++i) {
        if (i >= a.n_metrics) break;
        // (the copy was read from L2 after the ticket, so it holds what CTA 0 of this launch
        // may have just rewritten)
        if (!ks->has_thr[L][i]) { s_no_thr = 1; continue; }
        if (!((a.metric_mask >> i) & 1u)) continue;
        const double q2 = ks->thr[L][i][1];
        const double tau_lower = ks->thr[L][i][4], tau_upper = ks->thr[L][i][5];
        // (written so that a score that is not a number -- projections beyond the fp32 range --
        // counts as outside and never joins the history)
        const bool outside = !(g[i] >= tau_lower && g[i] <= tau_upper);
        if (outside) my_flag |= (1u << i);
        // ("x100 above the threshold", Sec. 3.1, is said of a deviation that broke the threshold: a
        // clean step never counts as severe, not even when the window is a single point)
        if (tid == 0 && outside && fabs(g[i] - q2) >= a.severe_mult * (tau_upper - q2)) s_severe = 1;
      }
    }
    s_flag[tid] = my_flag;
    if (ks) { ring_head = ks->hist_head[tid ? 1 : 0]; ring_count = ks->hist_count[tid ? 1 : 0]; }
  }
  const int any_flag = __syncthreads_or(my_flag != 0u);

  // Who joins the history: verified step, the units that raised nothing; warm-up, every unit
  // unless the input was non-finite (then nothing changes).
  const bool warmup_ok = (a.mode == kModeWarmup || a.mode == kModeReplicaWarmup) && !any_flag;
  if (tid < rows) {
    const bool joins = testing ? (my_flag == 0u) : warmup_ok;
    if (joins) {
      // the k-th unit of a level to join goes to ring slot (head + count + k) mod size; the
      // ring has `units` slots more than the window, so what is pushed out is not overwritten
      const int L = tid ? 1 : 0, size = ring_size(L ? a.cap1 : a.cap0, L ? a.units1 : a.units0);
      int k = 0;
      if (L && testing)
        for (int r = 1; r < tid; ++r) k += (s_flag[r] == 0u);
      else if (L)
        k = tid - 1;
      const int idx = (int)(((long long)ring_head + ring_count + k) % size);
#pragma unroll
      for (int i = 0; i < kNumMetrics; ++i)
        if (i < a.n_metrics && SENTINEL_BOUNDS(kSiteRing, ring_offset(L, i, a.cap0, a.cap1, a.units0, a.units1) + idx, 1, a.ring_doubles))
          a.hist[ring_offset(L, i, a.cap0, a.cap1, a.units0, a.units1) + idx] = g[i];
    }
    if (ft.scores_out) {
#pragma unroll
      for (int i = 0; i < kNumMetrics; ++i)
        if (i < a.n_metrics) ft.scores_out[tid * a.n_metrics + i] = (float)g[i];
    }
    if (a.stats_out) {                           // off the decision path
      const UnitSums &u = s_unit[tid];
      const double n = (tid == 0) ? (double)B * (double)Ns : (double)Ns;
      const double sq_x = fmax(u.s[1] + 2. * u.x0 * u.s[0] + n * u.x0 * u.x0, 0.);   // sum x^2
      const double sq_m = fmax(u.s[3] + 2. * u.m0 * u.s[2] + n * u.m0 * u.m0, 0.);
      double st[kNumStats] = {u.x0 + u.s[0] * inv_n, st_var_x, sqrt(sq_x), u.m0 + u.s[2] * inv_n,
                              st_var_m, st_cov, sqrt(sq_m), st_rho};
      for (int i = 0; i < kNumStats; ++i)
        a.stats_out[tid * kNumStats + i] = nonfinite ? CUDART_NAN_F : (float)st[i];
    }
  }

  if (tid == kDecider && a.mode != kModeDistance) {
    HandleState *hs = &s_hs;
    unsigned status = 0u;
    if (!replica || w == 0) {                    // an iteration starts with its first worker
      ks->steps += 1;
      ks->step_collected = ks->step_tainted = ks->step_nonfinite = ks->step_elsewhere = 0u;
    }
    int joined[2] = {0, 0};
    if (testing) {
      if (any_flag) {                            // violation counter with forgiveness, per worker
        hs->violations[w] += 1;
        hs->clean_streak[w] = 0;
        if (hs->violations[w] >= a.ban_violations || s_severe) hs->banned[w] = 1;
      } else {
        hs->clean_streak[w] += 1;
        if (hs->clean_streak[w] >= a.forgiveness_steps) {
          hs->violations[w] = hs->violations[w] > 0 ? hs->violations[w] - 1 : 0;
          hs->clean_streak[w] = 0;
        }
      }
      joined[0] = (s_flag[0] == 0u);
      for (int r = 1; r < rows; ++r) joined[1] += (s_flag[r] == 0u);
      ks->refresh_pending = 1;
      if (!replica) {
        ks->last_flagged = any_flag ? 1 : 0;
        if (!any_flag) {                         // m_t := candidate
          if (a.defer_commit) ks->commit_pending = 1; else ks->active ^= 1;
          status |= kFlagCommitted;
        }
      }
      if (s_severe) status |= kFlagSevere;
      if (hs->banned[w]) status |= kFlagBanned;
      if (s_no_thr) status |= kFlagNoThresholds;
    } else if (warmup_ok) {                      // warm-up: everything joins, always commit
      joined[0] = 1;
      joined[1] = B;
      ks->refresh_pending = 1;
      if (!replica) { if (a.defer_commit) ks->commit_pending = 1; else ks->active ^= 1; }
    }
    if (replica) {                               // what the mean over the clean workers needs
      ks->step_collected |= 1u << w;
      if (any_flag) ks->step_tainted |= 1u << w;
      if (s_flag[0] & kFlagNonfinite) ks->step_nonfinite |= 1u << w;
    }
    for (int L = 0; L < 2; ++L) {                // window bookkeeping after `joined` appends
      const int cap = L ? a.cap1 : a.cap0, size = ring_size(cap, L ? a.units1 : a.units0);
      const int total = ks->hist_count[L] + joined[L];
      const int evicted = total > cap ? total - cap : 0;
      ks->hist_count[L] = total - evicted;
      ks->hist_head[L] = (int)(((long long)ks->hist_head[L] + evicted) % size);
      // (several workers append between two refreshes: what the refresh merges accumulates)
      if (ks->refresh_pending) { ks->last_joined[L] += joined[L]; ks->last_evicted[L] += evicted; }
    }
    if (ft.last) s_hs.ticket = 0u;               // ready for the next launch
#ifdef SENTINEL_CHECK_BOUNDS
    if (*reinterpret_cast<volatile unsigned long long *>(&g_bounds_violations)) hs->error = kErrBounds;
#endif
    s_status = status;
  }
  __syncthreads();
  if (ft.flags_out && tid < rows)
    ft.flags_out[tid] = s_flag[tid] | (tid == 0 ? s_status : 0u);
  if (a.hs) {                                    // write the state back
    if (tid < kStateWords)
      reinterpret_cast<unsigned long long *>(a.hs)[tid] = reinterpret_cast<unsigned long long *>(&s_hs)[tid];
  } else if (tid == 0) {
    *a.ticket = 0u;
  }
}

// ---------------------------------------------------------------------------------------------
// kernels

// grid = 1 + G CTAs.  CTA 0 owes no rows: it brings the thresholds up to date (if the last
// step left that pending) while the others stream.  Every CTA then takes a ticket; whoever
// draws the last one has, by the fence/atomic order, everybody's partial sums and the fresh
// thresholds in view, and finalizes.  No CTA ever waits for another.
// (kScalar = true is the variant for rows of x that are strided or not 16-byte aligned, of any
// width; kShifted = true the one for such rows when the width is a multiple of 8: the vector
// path with x put in place by a funnel shift.  They are kernels of their own so that the vector
// path keeps its registers.  kBf16 = true: the reference buffers hold bf16 instead of fp32.)
template <bool kScalar, bool kBf16, bool kShifted = false>
__global__ void __launch_bounds__(kThreads)
stream_kernel_t(const StreamArgs a) {
  __shared__ unsigned long long s_part[kWarps][kSlotWords];
  __shared__ int s_last;
  extern __shared__ double s_dyn[];            // refresh_smem_doubles(cap0, cap1) when a handle is given

  // Programmatic dependent launch: let the next launch on the stream be set up while this one
  // runs, and do not touch memory before the previous launch has completed and flushed.  With
  // a plain launch both instructions do nothing.
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const void *m_in;
  void *m_out;
  if (a.mode == kModeDistance) {
    m_in = a.m_ext;
    m_out = nullptr;
  } else {
    const int act = __ldcg(&a.hs->kind[a.kind].active);   // written by an earlier launch only
    m_in = a.ema[act];
    m_out = a.ema[act ^ 1];
  }

  if (blockIdx.x == 0) {
    if (a.hs) {
      KindState *ks = &a.hs->kind[a.kind];
      if (ks->refresh_pending)
        refresh_thresholds(ks, a.hist, a.sorted, a.cap0, a.cap1, a.units0, a.units1, a.n_metrics, a.a5, s_dyn);
    }
  } else {
    stream_cta<kScalar, kBf16, kShifted>(a, blockIdx.x - 1, m_in, m_out, s_part);
  }

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned t = atomicAdd(a.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const FinalizeTarget ft = {0, a.partials, a.scores_out, a.flags_out, a.sw, 0, 1, 0};
  finalize(a, ft);
}

// ---------------------------------------------------------------------------------------------
// One [d] reference for all B*T tokens of a tensor (a reference reduced over samples and
// tokens): every token row is compared with the same vector m, and Eq. 1 moves m with the mean
// over the token rows, m' = beta m + (1-beta)/(B*T) sum_rows x[row, :].  Only x streams (2
// B/element); the work per element is what bounds the kernel.
//
// A CTA owns a block of rows as in the streaming kernel.  Inside, the columns are cut into
// stripes of 512 (a warp tile) and a warp keeps ONE stripe for all its rows: its tile of m stays
// in registers, and so do the column sums of x that Eq. 1 needs.  With fewer stripes than warps
// several warps share a stripe and take every wps-th row (`phases`); with more, a warp does
// several stripes one after the other.  Each (stripe, phase) pair is a slot: its column sums go
// to the CTA's block of `col_part`, and channel_mean_kernel adds the blocks up in a fixed order.
constexpr int kStripe = 8 * 32 * kUnroll;        // columns per stripe
constexpr int kChanThreads = 512;                 // threads per CTA of channel_ref_kernel: 16 warps, a stripe each at d = 8192
constexpr int kChanWarps = kChanThreads / 32;
constexpr int kChanRows = 6;                      // rows of a stripe that one stage holds
constexpr int kChanDepth = 2;                     // stages per warp

__host__ __device__ inline int channel_stripes(int d) { return (d + kStripe - 1) / kStripe; }
__host__ __device__ inline int channel_phases(int d) {
  const int stripes = channel_stripes(d);
  return stripes < kChanWarps ? kChanWarps / stripes : 1;
}
__host__ __device__ inline int channel_slots(int d) { return channel_stripes(d) * channel_phases(d); }

// a warp's part of the dynamic shared memory: its ring of stages (kChanRows rows of its stripe,
// 1 KB each, filled by bulk copies two stages ahead of the arithmetic) and their barriers
struct __align__(128) ChanWarp {
  unsigned char stage[kChanDepth][kChanRows * kTileBytesX];
  unsigned long long bar[kChanDepth];
};
__host__ __device__ inline size_t channel_smem_bytes() { return (size_t)kChanWarps * sizeof(ChanWarp); }

// what a warp carries from slot to slot
struct ChanState {
  unsigned stages_done;      // stages this warp has consumed since the launch: stage index and barrier phase follow from it
  bool alive;                // false once a wait gave up
};

// Exact zeros of the staged rows whose sign bit equals that of m (the packed sign test did not
// count them), and non-finite elements: the two rare looks at a stage, kept out of line.
__device__ __noinline__ unsigned channel_uncounted_zeros(const unsigned char *stage, int rows, int lane, unsigned valid,
                                                         const float *m_stripe) {
  unsigned n = 0u;
  for (int i = 0; i < rows; ++i)
    for (int u = 0; u < kUnroll; ++u) {
      if (!((valid >> u) & 1u)) continue;
      const uint16_t *xw = reinterpret_cast<const uint16_t *>(stage + i * kTileBytesX + (size_t)(u * 32 + lane) * 16);
      const float *mw = m_stripe + (size_t)(u * 32 + lane) * 8;
      for (int e = 0; e < 8; ++e) {
        const unsigned xb = xw[e];
        if ((xb & 0x7FFFu) == 0u && (xb >> 15) == (__float_as_uint(__ldg(mw + e)) >> 31)) ++n;
      }
    }
  return n;
}
__device__ __noinline__ unsigned channel_nonfinite_in_stage(const unsigned char *stage, int rows, int lane, unsigned valid) {
  unsigned nf = 0u;
  for (int i = 0; i < rows; ++i)
    for (int u = 0; u < kUnroll; ++u) {
      if (!((valid >> u) & 1u)) continue;
      const uint4 w = *reinterpret_cast<const uint4 *>(stage + i * kTileBytesX + (size_t)(u * 32 + lane) * 16);
      nf |= (((w.x & 0x7F807F80u) + 0x00800080u) | ((w.y & 0x7F807F80u) + 0x00800080u) |
             ((w.z & 0x7F807F80u) + 0x00800080u) | ((w.w & 0x7F807F80u) + 0x00800080u)) & 0x80008000u;
    }
  return nf;
}

__device__ __noinline__ unsigned channel_differs_in_stage(const unsigned char *stage, int rows, int lane, unsigned valid,
                                                          unsigned x0pair) {
  unsigned diff = 0u;
  for (int i = 0; i < rows; ++i)
    for (int u = 0; u < kUnroll; ++u) {
      if (!((valid >> u) & 1u)) continue;
      const uint4 w = *reinterpret_cast<const uint4 *>(stage + i * kTileBytesX + (size_t)(u * 32 + lane) * 16);
      diff |= (w.x ^ x0pair) | (w.y ^ x0pair) | (w.z ^ x0pair) | (w.w ^ x0pair);
    }
  return diff;
}

// One slot (a warp's stripe of columns, every `phases`-th row from `first` on) of a segment.
// Per element only what is not linear in x is done: (x - x0)^2, |x - m|, the sign test on the
// packed pairs, the constancy bits, and the column sum of x - x0.  The linear sums follow from
// the column sums when the slot is done: sum (x - x0) = sum_c col_c and sum (x - x0)(m - m0) =
// sum_c (m_c - m0) col_c, since m is the same in every row.  Non-finite elements show in the sum
// of |x - m| (not a finite number then), exact zeros of x in the packed minimum: either is looked
// at once per stage, and the stage is gone through again only if it shows.
// kZeroInM = true (an exact zero among this warp's columns of m): the general sign test.
template <bool kZeroInM, bool kFull>
__device__ __forceinline__ void channel_slot(const uint16_t *xslot, size_t row_pitch, int n_rows, int vc,
                                             const bool (&ok)[kUnroll], const F8 (&mv)[kUnroll],
                                             const unsigned (&msp)[kUnroll][4], const float *m_stripe,
                                             float (&cs)[kUnroll][8], unsigned x0pair, float x0f, ThreadAcc &t,
                                             ChanWarp &cw, ChanState &st, long long x_first, long long x_extent) {
  // (xslot: the first element of the stripe in the slot's first row; rows are row_pitch elements apart)
  const int lane = threadIdx.x & 31;
  const int n_stages = (n_rows + kChanRows - 1) / kChanRows;
  const unsigned valid = (ok[0] ? 1u : 0u) | (ok[1] ? 2u : 0u);
  static_assert(kUnroll == 2, "two chunks per lane and row");
  // the ring is addressed by the warp's running stage count, so that barrier phases carry on
  // from slot to slot; `head` = count at which this slot's stage 0 is consumed
  const unsigned head = st.stages_done;
  auto fill = [&](int s) {
    if (s < n_stages && lane == 0) {
      const int rows = (n_rows - s * kChanRows < kChanRows) ? n_rows - s * kChanRows : kChanRows;
      const unsigned k = head + (unsigned)s, slot = k % kChanDepth;
      const unsigned bar = smem_addr(&cw.bar[slot]), dst = smem_addr(&cw.stage[slot][0]);
      // (checked build: the last element of the stage's last row must lie in x)
      if (SENTINEL_BOUNDS(kSiteStageX, x_first + (long long)(s * kChanRows + rows - 1) * (long long)row_pitch, (long long)vc * 8, x_extent) &&
          SENTINEL_BOUNDS(kSiteStageX, x_first + (long long)(s * kChanRows) * (long long)row_pitch, (long long)vc * 8, x_extent)) {
        mbar_arrive_expect(bar, (unsigned)(rows * vc) * 16u);
        for (int i = 0; i < rows; ++i)
          bulk_copy_in(dst + i * kTileBytesX, xslot + (size_t)(s * kChanRows + i) * row_pitch, (unsigned)vc * 16u, bar);
      } else {
        mbar_arrive_expect(bar, 0u);
      }
    }
  };
#pragma unroll
  for (int s = 0; s < kChanDepth; ++s) fill(s);

  for (int s = 0; s < n_stages; ++s) {
    const unsigned k = head + (unsigned)s, slot = k % kChanDepth;
    if (!__all_sync(0xffffffffu, mbar_wait(smem_addr(&cw.bar[slot]), (k / kChanDepth) & 1u))) {
      // the stage never arrived: wait out what else is in flight, then give up on the warp's rows
      for (int q = 1; q < kChanDepth; ++q)
        if (s + q < n_stages) mbar_wait(smem_addr(&cw.bar[(k + q) % kChanDepth]), ((k + q) / kChanDepth) & 1u);
      st.alive = false;
      st.stages_done = k;                                    // (nothing is issued any more)
      return;
    }
    const unsigned char *stage = cw.stage[slot];
    const int rows = (n_rows - s * kChanRows < kChanRows) ? n_rows - s * kChanRows : kChanRows;
    F2 g_sxx2[kUnroll] = {{0.f, 0.f}, {0.f, 0.f}};             // (several chains: the adds of a row do not wait for one another)
    float g_ab[kUnroll] = {0.f, 0.f};
    unsigned flips = 0u, zmin = 0x7F7F7F7Fu;
#pragma unroll 2
    for (int i = 0; i < rows; ++i) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        if (!kFull && !ok[u]) continue;
        const uint4 w = *reinterpret_cast<const uint4 *>(stage + i * kTileBytesX + (size_t)(u * 32 + lane) * 16);
        const unsigned w4[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (!kZeroInM) {
            flips = __dp4a((w4[q] ^ msp[u][q]) & 0x80008000u, 0x01010101u, flips);
            zmin = min_abs_bf16x2(zmin, w4[q]);
          }
          const F2 xf = {__uint_as_float(w4[q] << 16), __uint_as_float(w4[q] & 0xFFFF0000u)};
          const F2 mf = {mv[u].v[2 * q], mv[u].v[2 * q + 1]};
          const F2 xs = sub2(xf, F2{x0f, x0f});
          const F2 df = sub2(xf, mf);
          g_sxx2[u] = fma2(xs, xs, g_sxx2[u]);
          g_ab[u] += fabsf(df.lo);
          g_ab[u] += fabsf(df.hi);
          const F2 c2 = add2(F2{cs[u][2 * q], cs[u][2 * q + 1]}, xs);
          cs[u][2 * q] = c2.lo;
          cs[u][2 * q + 1] = c2.hi;
          if (kZeroInM) {
            const unsigned xl = __float_as_uint(xf.lo) ^ (__float_as_uint(mf.lo) & 0x80000000u);
            const unsigned xh = __float_as_uint(xf.hi) ^ (__float_as_uint(mf.hi) & 0x80000000u);
            flips += (((xf.lo == 0.f) != (mf.lo == 0.f)) || (__uint_as_float(xl) < 0.f)) ? kFlipUnit : 0u;
            flips += (((xf.hi == 0.f) != (mf.hi == 0.f)) || (__uint_as_float(xh) < 0.f)) ? kFlipUnit : 0u;
          }
        }
      }
    }
    if (!kZeroInM && __any_sync(0xffffffffu, ((zmin & 0x7FFFu) == 0u) || ((zmin & 0x7FFF0000u) == 0u)))
      flips += kFlipUnit * channel_uncounted_zeros(stage, rows, lane, valid, m_stripe);
    if (__any_sync(0xffffffffu, !(g_ab[0] + g_ab[1] <= 3.4028234664e38f)))
      t.nf_bits |= channel_nonfinite_in_stage(stage, rows, lane, valid);
    // does x vary?  A non-zero sum of (x - x0)^2 says so; a lane whose sum is zero (all its elements
    // equal to x0, or differences too small to square) has its bit patterns compared
    const float g_sxx[kUnroll] = {g_sxx2[0].lo + g_sxx2[0].hi, g_sxx2[1].lo + g_sxx2[1].hi};
    if (g_sxx[0] + g_sxx[1] > 0.f) t.x_diff |= 1u;
    if (__any_sync(0xffffffffu, !(g_sxx[0] + g_sxx[1] > 0.f)))
      t.x_diff |= channel_differs_in_stage(stage, rows, lane, valid, x0pair);
    t.sxx += (double)g_sxx[0] + (double)g_sxx[1];            // the short fp32 runs into the fp64 sums
    t.ab += (double)g_ab[0] + (double)g_ab[1];
    t.flips += flips / kFlipUnit;
    // every lane has used what it read from the stage (the sums above depend on it): refill it
    __syncwarp();
    fill(s + kChanDepth);
  }
  st.stages_done = head + (unsigned)n_stages;
}

// (merge: the column sums are added to what the CTA's first segment left in col_seg instead of
// replacing it -- one vector for all samples needs no separation by sample)
__device__ void channel_segment(const StreamArgs &a, int b, long long ra, long long rb, const float *m_in,
                                float *col_seg, bool merge, ChanWarp &cw, ChanState &st,
                                unsigned long long (*s_part)[kSlotWords], unsigned long long *slot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = a.d >> 3;                   // d is a multiple of 8 here
  const int stripes = channel_stripes(a.d), phases = channel_phases(a.d), n_slots = stripes * phases;
  const unsigned x0 = a.x[(size_t)b * a.T * (size_t)a.d];
  const unsigned x0pair = x0 | (x0 << 16);
  const float x0f = __uint_as_float(x0 << 16);
  const unsigned m0bits = __float_as_uint(__ldg(m_in));
  const float m0 = __uint_as_float(m0bits);
  const int seg_rows = (int)(rb - ra);

  ThreadAcc t = {0., 0., 0., 0., 0., 0., 0u, 0u, 0u, 0u};
  for (int sl = warp; sl < n_slots; sl += kChanWarps) {
    const int stripe = sl % stripes, phase = sl / stripes;
    bool ok[kUnroll];
    F8 mv[kUnroll];                              // this lane's 8 + 8 columns of the reference
    unsigned msp[kUnroll][4];                    // their sign bits, per pair at bits 15 and 31
    float cs[kUnroll][8];                        // column sums of x - x0 over the slot's rows
    float lm = 0.f, lmm = 0.f;                   // this lane's sums of (m - m0), (m - m0)^2 over its columns
    unsigned m_diff = 0u;
    bool zero_in_m = false;
    int vc = chunks - stripe * 32 * kUnroll;     // chunks of this stripe that exist
    if (vc > 32 * kUnroll) vc = 32 * kUnroll;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int c = stripe * 32 * kUnroll + u * 32 + lane;
      ok[u] = c < chunks && SENTINEL_BOUNDS(kSiteRefIn, (long long)c * 8, 8, a.d);
#pragma unroll
      for (int e = 0; e < 8; ++e) { cs[u][e] = 0.f; mv[u].v[e] = 1.f; }
      if (ok[u]) {
        const float4 *mp = reinterpret_cast<const float4 *>(m_in) + (size_t)c * 2;
        const float4 lo = __ldg(mp), hi = __ldg(mp + 1);
        mv[u].v[0] = lo.x; mv[u].v[1] = lo.y; mv[u].v[2] = lo.z; mv[u].v[3] = lo.w;
        mv[u].v[4] = hi.x; mv[u].v[5] = hi.y; mv[u].v[6] = hi.z; mv[u].v[7] = hi.w;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float ms = mv[u].v[e] - m0;
          lm += ms;
          lmm = fmaf(ms, ms, lmm);
          m_diff |= __float_as_uint(mv[u].v[e]) ^ m0bits;
          zero_in_m |= (mv[u].v[e] == 0.f);
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        msp[u][q] = __byte_perm(__float_as_uint(mv[u].v[2 * q]), __float_as_uint(mv[u].v[2 * q + 1]), 0x7733);
    }
    const int n_rows = (seg_rows - phase + phases - 1) / phases;      // rows phase, phase + phases, ... of the segment
    const uint16_t *xslot = a.x + (size_t)(ra + phase) * a.d + (size_t)stripe * kStripe;
    const float *m_stripe = m_in + (size_t)stripe * kStripe;
    if (st.alive && n_rows > 0) {
      const bool full = vc == 32 * kUnroll;              // every lane has both its chunks
      if (__any_sync(0xffffffffu, zero_in_m))              // (rare: the reference starts out as all zeros)
        channel_slot<true, false>(xslot, (size_t)phases * a.d, n_rows, vc, ok, mv, msp, m_stripe, cs, x0pair, x0f, t, cw, st, (long long)(xslot - a.x), a.x_extent);
      else if (full)
        channel_slot<false, true>(xslot, (size_t)phases * a.d, n_rows, vc, ok, mv, msp, m_stripe, cs, x0pair, x0f, t, cw, st, (long long)(xslot - a.x), a.x_extent);
      else
        channel_slot<false, false>(xslot, (size_t)phases * a.d, n_rows, vc, ok, mv, msp, m_stripe, cs, x0pair, x0f, t, cw, st, (long long)(xslot - a.x), a.x_extent);
    }

    // what is linear in x, from the column sums; the reference's own sums: its columns once per row
    float4 *dst = reinterpret_cast<float4 *>(col_seg + (size_t)sl * kStripe) + lane * 2;
    const bool col_ok = SENTINEL_BOUNDS(kSiteColumns, (col_seg - a.col_part) + (long long)(sl + 1) * kStripe, 0, a.col_floats);
    double s_x = 0., s_xm = 0.;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float4 lo = make_float4(cs[u][0], cs[u][1], cs[u][2], cs[u][3]);
      float4 hi = make_float4(cs[u][4], cs[u][5], cs[u][6], cs[u][7]);
      if (merge && col_ok) {                     // (written by this very lane while it did the first segment)
        const float4 plo = dst[u * 64], phi = dst[u * 64 + 1];
        lo.x += plo.x; lo.y += plo.y; lo.z += plo.z; lo.w += plo.w;
        hi.x += phi.x; hi.y += phi.y; hi.z += phi.z; hi.w += phi.w;
      }
      if (col_ok) {
        dst[u * 64] = lo;
        dst[u * 64 + 1] = hi;
      }
      if (ok[u]) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          s_x += (double)cs[u][e];
          s_xm += (double)(mv[u].v[e] - m0) * (double)cs[u][e];
        }
      }
    }
    t.sx += s_x;
    t.sxm += s_xm;
    const int rows_done = (n_rows > 0) ? n_rows : 0;
    t.sm += (double)rows_done * (double)lm;
    t.smm += (double)rows_done * (double)lmm;
    if (rows_done) t.m_diff |= m_diff;
  }
  reduce_to_slot(t, b, x0, m0bits, s_part, slot);
}

// (kPerSample: a vector per sample, [B,d], instead of one, [d]; a kernel of its own so that the
// code of either form does not depend on the other's addressing)
template <bool kPerSample>
__global__ void __launch_bounds__(kChanThreads)
channel_ref_kernel(const StreamArgs a) {
  __shared__ unsigned long long s_part[kWarps][kSlotWords];
  __shared__ int s_last;
  extern __shared__ __align__(128) double s_dyn[];   // CTA 0: the refresh's working copies; the others: the warps' staging rings

  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int act = __ldcg(&a.hs->kind[a.kind].active);     // written by an earlier launch only
  const float *m_in = static_cast<const float *>(a.ema[act]);

  if (blockIdx.x == 0) {
    KindState *ks = &a.hs->kind[a.kind];
    if (ks->refresh_pending)
      refresh_thresholds(ks, a.hist, a.sorted, a.cap0, a.cap1, a.units0, a.units1, a.n_metrics, a.a5, s_dyn);
  } else {
    const int c = blockIdx.x - 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    ChanWarp &cw = reinterpret_cast<ChanWarp *>(s_dyn)[warp];
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < kChanDepth; ++k) mbar_init(smem_addr(&cw.bar[k]), 1u);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    ChanState st = {0u, true};
    const long long R = (long long)a.B * a.T;
    const long long R0 = (R * c) / a.G, R1 = (R * (c + 1)) / a.G;
    const size_t seg_floats = (size_t)channel_slots(a.d) * kStripe;
    long long ra = R0;
    for (int sgm = 0; sgm < kSegsPerCta; ++sgm) {
      unsigned long long *slot = a.partials + ((size_t)c * kSegsPerCta + sgm) * kSlotWords;
      // column sums: a block per (CTA, segment) with a vector per sample, one block per CTA (both
      // segments added) with one vector for all
      const bool merge = !kPerSample && sgm > 0;
      float *col_seg = a.col_part + ((size_t)c * kSegsPerCta + (kPerSample ? sgm : 0)) * seg_floats;
      if (ra < R1) {
        const int b = (int)(ra / a.T);
        const long long sample_end = (long long)(b + 1) * a.T;
        const long long rb = sample_end < R1 ? sample_end : R1;
        channel_segment(a, b, ra, rb, kPerSample ? m_in + (size_t)b * a.d : m_in, col_seg, merge, cw, st, s_part, slot);
        ra = rb;
      } else {                                    // no rows: nothing to add
        if (kPerSample)
          for (size_t i = threadIdx.x; i < seg_floats; i += kChanThreads) col_seg[i] = 0.f;
        if (threadIdx.x == 0) slot[7] = 0ull;
      }
    }
    if (!st.alive && lane == 0) atomicExch(&a.hs->error, kErrStagingTimeout);
  }

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned t = atomicAdd(a.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const FinalizeTarget ft = {0, a.partials, a.scores_out, a.flags_out, nullptr, 0, 1, 0};
  finalize(a, ft);
}

// Second half of a step with a [d] reference: if the step committed, Eq. 1 with the mean over
// the token rows into the spare buffer; the last CTA then makes that buffer the reference.  The
// streaming CTAs left column sums of x - x0 per (CTA, segment, slot), x0 the first element of the
// segment's sample; they are added in a fixed order, in double precision -- a CTA takes 32
// columns, its 16 groups of threads every 16th block of partial sums -- and the shifts come back as
// the one constant T * sum_b x[b,0,0].
constexpr int kChannelMeanCols = 32, kChannelMeanGroups = 16;

__global__ void __launch_bounds__(kChannelMeanCols * kChannelMeanGroups)
channel_mean_kernel(HandleState *hs, int kind, float *ema0, float *ema1, const float *col_part, const uint16_t *x,
                    int G, int B, int T, int d, int per_sample, float beta, float one_minus_beta) {
  __shared__ double s_sum[kChannelMeanGroups][kChannelMeanCols];
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  KindState *ks = &hs->kind[kind];
  // (cleared only by the CTA that draws the last ticket, i.e. after every CTA has read it)
  if (!__ldcg(&ks->commit_pending)) return;
  const int act = __ldcg(&ks->active);
  // blockIdx.y: with a vector per sample, the sample whose vector this CTA moves
  const int sample = per_sample ? (int)blockIdx.y : -1;
  const size_t ref_off = per_sample ? (size_t)sample * d : 0;
  const float *m_in = (act ? ema1 : ema0) + ref_off;
  float *m_out = (act ? ema0 : ema1) + ref_off;
  const int lane_c = threadIdx.x % kChannelMeanCols, group = threadIdx.x / kChannelMeanCols;
  const int c = blockIdx.x * kChannelMeanCols + lane_c;
  const int stripes = channel_stripes(d), phases = channel_phases(d), n_slots = stripes * phases;
  const long long R = (long long)B * T;
  // (CTA, segment) pairs whose blocks of partial sums can belong to this vector: all of them, or
  // with a vector per sample the CTAs whose rows [R*cta/G, R*(cta+1)/G) can touch the sample's
  // (a superset; the test in the loop decides)
  int cs_lo = 0, cs_hi = G * kSegsPerCta;
  if (per_sample) {
    long long lo = ((long long)sample * T * G) / R - 1, hi = ((long long)(sample + 1) * T * G + R - 1) / R + 1;
    if (lo < 0) lo = 0;
    if (hi > G) hi = G;
    cs_lo = (int)lo * kSegsPerCta;
    cs_hi = (int)hi * kSegsPerCta;
  }
  double sum = 0.;
  if (c < d) {
    const int stripe = c / kStripe, within = c - stripe * kStripe;
    const float *src = col_part + (size_t)stripe * kStripe + within;
    if (!per_sample) {                         // one block per CTA: its first, with both segments added
#pragma unroll 8
      for (int i = group; i < G * phases; i += kChannelMeanGroups) {
        const int cta = i / phases, p = i - cta * phases;  // CTA and row phase
        sum += (double)__ldcg(src + ((size_t)cta * kSegsPerCta * n_slots + (size_t)p * stripes) * kStripe);
      }
    } else {
      for (int i = cs_lo * phases + group; i < cs_hi * phases; i += kChannelMeanGroups) {
        const int cs = i / phases, p = i - cs * phases;
        // a CTA's first segment lies in the sample of its first row, floor(floor(B*T*cta/G) / T) =
        // floor(B*cta/G), its second (if any: else blocks of zeros) in the next one
        if ((B * (cs >> 1)) / G + (cs & 1) != sample) continue;
        sum += (double)__ldcg(src + ((size_t)cs * n_slots + (size_t)p * stripes) * kStripe);
      }
    }
  }
  s_sum[group][lane_c] = sum;
  __syncthreads();
  if (group == 0 && c < d) {
    double total = 0., shift = 0.;
    for (int g = 0; g < kChannelMeanGroups; ++g) total += s_sum[g][lane_c];
    for (int b = per_sample ? sample : 0; b < (per_sample ? sample + 1 : B); ++b)
      shift += (double)__uint_as_float((unsigned)x[(size_t)b * T * (size_t)d] << 16);
    const double rows = per_sample ? (double)T : (double)B * (double)T;
    m_out[c] = (float)((double)beta * (double)m_in[c] + (double)one_minus_beta * ((total + (double)T * shift) / rows));
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned tk = atomicAdd(&hs->ticket2, 1u);
    if (tk == gridDim.x * gridDim.y - 1) {
      __threadfence();
      ks->active = act ^ 1;
      ks->commit_pending = 0;
      hs->ticket2 = 0u;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// All workers of a stage in one launch (worker loop of Alg. 2 / Alg. 3, Alg. 1 main loop).
//
// Every worker's tensor is tested against the same m_{t-1}, so a tile of m is loaded once and
// each worker's tile of x is streamed past it: 2 B per worker and element plus 4 B of m read and
// 4 B written, instead of a pass over m per worker and another over every x for the mean.  The
// write is the mean over all collected workers, m' = beta m + (1-beta)/n sum_r x^(r), put into
// the spare buffer on the assumption that nobody will be flagged; the last CTA scores the workers
// one after the other (pooled history, per-worker counters) and, if indeed nobody was flagged,
// makes that buffer the reference.  Otherwise the mean over the clean workers is taken afterwards
// by ema_mean_kernel from the untouched m_{t-1}.
//
// A thread cannot carry fp64 sums for 16 workers, so after every warp tile (512 elements) the
// tile's fp32 sums are added up across the warp and one lane folds them into the warp's fp64
// accumulators in shared memory.
struct ReplicaArgs {
  StreamArgs s;                       // x, scores_out, flags_out, sw unused
  const uint16_t *xs[kMaxWorkers];    // worker r's tensor; not read for a worker in tainted_in
  unsigned long long *partials;       // [R][G][2][kSlotWords]
  float *scores_all;                  // [R][(1+B)*n_metrics]
  unsigned *flags_all;                // [R][1+B] or nullptr (warm-up)
  const float *sw_all;                // [R][1+B] sliced Wasserstein distances, or nullptr
  unsigned tainted_in;                // bit r: worker r was tainted at another stage
  int pad;
};

struct ReplicaShared {
  double acc[kWarps][kMaxWorkers][4];             // sums of (x-x0), (x-x0)^2, (x-x0)(m-m0), |x-m|
  unsigned long long flips[kWarps][kMaxWorkers];
  unsigned bits[kWarps][kMaxWorkers];             // kBitNonfinite | kBitXVaries
  double m_acc[kWarps][2];                        // sums of (m-m0), (m-m0)^2
  unsigned m_varies[kWarps];
  unsigned x0[kMaxWorkers];                       // the sample's first element, per worker
};

// One tensor's tile against the tile of m.  kZeroInM = false is the usual case, no exact zero in
// the warp's tile of m (found out once per tile, for all tensors that share it): then
// sign(x) != sign(m) iff x, with its sign bit flipped where m is negative, is <= +0 as an integer
// (a negative number, -0, or +0: x and m differ in sign, or x is zero against a non-zero m).
template <bool kZeroInM>
__device__ __forceinline__ void replica_tile(const uint4 (&cur)[kUnroll], const F8 (&mv)[kUnroll], const bool (&ok)[kUnroll],
                                             float x0f, float m0, unsigned x0pair, float (&sum)[kUnroll][8], float &sx,
                                             float &sxx, float &sxm, float &ab, unsigned &flips, unsigned &nf,
                                             unsigned &x_diff) {
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    if (!ok[u]) continue;
    const unsigned w4[4] = {cur[u].x, cur[u].y, cur[u].z, cur[u].w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      nf |= ((w4[q] & 0x7F807F80u) + 0x00800080u) & 0x80008000u;
      x_diff |= w4[q] ^ x0pair;
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        const float xf = __uint_as_float(hlf ? (w4[q] & 0xFFFF0000u) : (w4[q] << 16));
        const float mf = mv[u].v[2 * q + hlf];
        const float xs = xf - x0f, ms = mf - m0;
        sx += xs;
        sxx = fmaf(xs, xs, sxx);
        sxm = fmaf(xs, ms, sxm);
        ab += fabsf(xf - mf);
        const unsigned xt = __float_as_uint(xf) ^ (__float_as_uint(mf) & 0x80000000u);
        if (kZeroInM) flips += (((xf == 0.f) != (mf == 0.f)) || (__uint_as_float(xt) < 0.f)) ? 1u : 0u;
        else flips += ((int)xt <= 0) ? 1u : 0u;
        sum[u][2 * q + hlf] += xf;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Up to kFewSets tensors against the tile of m: sums in registers, tiles staged by bulk copies.
//
// The general path below reduces each tile's sums across the warp and folds them into shared
// fp64 accumulators, once per tensor and tile: a third of its instructions.  With few tensors a
// thread keeps its own fp32 sums per tensor over kFoldTiles tiles (128 elements per tensor: the
// rounding of so short a run stays below 1e-6 of the sum, and the runs are many), after which
// the warp adds them up and folds them into its fp64 accumulators in shared memory; the warps are
// added up once, when the CTA's rows are done, in a fixed order.  Non-finite elements are found
// through the sum of |x - m|: it is not a finite number as soon as one x is not, so the exact
// test of the exponent bits runs only for a tile after which that sum is not finite.
//
// Each warp owns a two-stage ring in shared memory.  A stage holds one warp tile of the
// reference (2 KB) and the same tile of every tensor (1 KB each); one lane fills it with bulk
// asynchronous copies (cp.async.bulk, completion counted in bytes on the stage's mbarrier) two
// tiles ahead of the arithmetic, so that a tile's worth of bytes per warp is in flight the
// whole time without a register being held for it.  The warp that waits on a stage is the one
// that filled it; a wait that does not end (it always should) gives up after kStageWaitNs,
// records kErrStagingTimeout in the handle and skips the warp's remaining tiles.
constexpr int kFewSets = 4;
constexpr int kFoldTiles = 8;
constexpr int kFewThreads = 512;                  // threads per CTA of the kernels that take this path
constexpr int kFewWarps = kFewThreads / 32;
constexpr int kStageDepth = 2;
constexpr int kStageBytes = kTileBytesM + kFewSets * kTileBytesX;

// A CTA's rows lie in one sample or straddle one boundary: two segments, each with its own shift
// values, sums and slot.  A warp's tiles come in ascending row order, so it crosses over once.
struct FewShared {
  const uint16_t *ptr[kFewSets];                  // the tensors that stream, in order
  int widx[kFewSets];                             // which worker / sample each of them is (its slot block)
  unsigned x0[kSegsPerCta][kFewSets];             // the sample's first element, per segment and tensor
  unsigned m0bits[kSegsPerCta];                   // the sample's first element of the reference
  unsigned flips[kSegsPerCta][kFewWarps][kFewSets];
  unsigned bits[kSegsPerCta][kFewWarps][kFewSets];   // kBitNonfinite | kBitXVaries
  unsigned m_varies[kSegsPerCta][kFewWarps];
  int timed_out;
};
struct __align__(128) FewWarp {                   // a warp's part of the dynamic shared memory
  unsigned char stage[kStageDepth][kStageBytes];
  double acc[kSegsPerCta][kFewSets * 4 + 2];      // per tensor sums of (x-x0), (x-x0)^2, (x-x0)(m-m0), |x-m|; then of (m-m0), (m-m0)^2
  unsigned long long bar[kStageDepth];
};
__host__ __device__ inline size_t few_smem_bytes() { return (size_t)kFewWarps * sizeof(FewWarp); }

// One tensor's 8-element chunk against the chunk of m.  Sign mismatches are counted in units of
// kFlipUnit.  kZeroInM = true: the general three-valued sign test, element by element.
// kZeroInM = false (no exact zero in this chunk of m, the usual case): on the packed pairs --
// msp holds the sign bits of the two m's of a pair at bits 15 and 31, so (w ^ msp) & 0x80008000
// has a bit set per element whose sign bit differs from m's, and a byte-wise dot product with
// ones adds them up (0x80 each).  That is the mismatch count unless x holds an exact zero (a
// zero counts as a mismatch whatever its sign bit): zmin follows the smallest magnitude of the
// tensor's tile, and the caller corrects the count of a tile in which it reached zero.
template <bool kZeroInM>
__device__ __forceinline__ void few_chunk(const uint4 &cur, const F8 &mv, const unsigned (&msp)[4], float x0f, float m0,
                                          unsigned x0pair, float (&sum)[8], float &sx, float &sxx, float &sxm,
                                          float &ab, unsigned &flips, unsigned &x_diff, unsigned &zmin) {
  const unsigned w4[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    x_diff |= w4[q] ^ x0pair;
    if (!kZeroInM) {
      flips = __dp4a((w4[q] ^ msp[q]) & 0x80008000u, 0x01010101u, flips);
      zmin = min_abs_bf16x2(zmin, w4[q]);
    }
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
      const float xf = __uint_as_float(hlf ? (w4[q] & 0xFFFF0000u) : (w4[q] << 16));
      const float mf = mv.v[2 * q + hlf];
      const float xs = xf - x0f, ms = mf - m0;
      sx += xs;
      sxx = fmaf(xs, xs, sxx);
      sxm = fmaf(xs, ms, sxm);
      ab += fabsf(xf - mf);
      if (kZeroInM) {
        const unsigned xt = __float_as_uint(xf) ^ (__float_as_uint(mf) & 0x80000000u);
        flips += (((xf == 0.f) != (mf == 0.f)) || (__uint_as_float(xt) < 0.f)) ? kFlipUnit : 0u;
      }
      sum[2 * q + hlf] += xf;
    }
  }
}

// The two rare corrections of a tile, kept out of line so that they cost the streaming loop no
// registers.  `valid` = this lane's chunks (bit u) that exist.
// Exponent bits of all ones (NaN or infinity) among this lane's elements of tensor r's tile?
__device__ __noinline__ unsigned few_nonfinite_in_tile(const unsigned char *stage, int r, int lane, unsigned valid) {
  unsigned nf = 0u;
  for (int u = 0; u < kUnroll; ++u) {
    if (!((valid >> u) & 1u)) continue;
    const uint4 w = *reinterpret_cast<const uint4 *>(stage + kTileBytesM + r * kTileBytesX + (size_t)(u * 32 + lane) * 16);
    nf |= (((w.x & 0x7F807F80u) + 0x00800080u) | ((w.y & 0x7F807F80u) + 0x00800080u) |
           ((w.z & 0x7F807F80u) + 0x00800080u) | ((w.w & 0x7F807F80u) + 0x00800080u)) & 0x80008000u;
  }
  return nf;
}
// Exact zeros of tensor r whose sign bit equals that of m, in the chunks where the packed sign
// test ran (it did not count them): each is a mismatch all the same.  Returns their number.
// (ref_bf16: the staged tile of the reference holds bf16)
__device__ __noinline__ unsigned few_uncounted_zeros(const unsigned char *stage, int r, int lane, unsigned valid,
                                                     int ref_bf16) {
  unsigned n = 0u;
  for (int u = 0; u < kUnroll; ++u) {
    if (!((valid >> u) & 1u)) continue;
    const uint16_t *xw = reinterpret_cast<const uint16_t *>(stage + kTileBytesM + r * kTileBytesX + (size_t)(u * 32 + lane) * 16);
    const unsigned *mw = reinterpret_cast<const unsigned *>(stage + (size_t)(u * 32 + lane) * 32);
    const uint16_t *mh = reinterpret_cast<const uint16_t *>(stage + (size_t)(u * 32 + lane) * 16);
    for (int e = 0; e < 8; ++e) {
      const unsigned xb = xw[e];
      const unsigned m_sign = ref_bf16 ? (unsigned)(mh[e] >> 15) : (mw[e] >> 31);
      if ((xb & 0x7FFFu) == 0u && (xb >> 15) == m_sign) ++n;
    }
  }
  return n;
}

// Rows [r0, r1) of the flat [rows, d] view, of which [r0, cut) lie in sample b0 and [cut, r1) in
// sample b0 + 1 (cut = r1: one segment).  kFull: d is a multiple of the warp tile, no ragged tile.
// kBf16: the reference buffers hold bf16 (its tile is staged as 1 KB, widened when read, and the
// candidate is rounded to nearest even when stored).
template <int NR, bool kFull, bool kBf16>
__device__ void few_rows(const StreamArgs &a, unsigned long long *partials, int b0, long long r0, long long cut,
                         long long r1, const void *m_in, void *m_out, int c, FewShared &fs, FewWarp *fw_all) {
  constexpr unsigned kRefChunkBytes = kBf16 ? 16u : 32u;     // a lane's 8 elements of the reference
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunks = a.d >> 3;                               // d is a multiple of 8 here
  const int tiles_per_row = (chunks + 32 * kUnroll - 1) / (32 * kUnroll);
  const int n_tiles = (int)(r1 - r0) * tiles_per_row;
  const int cut_rr = (int)(cut - r0);                        // first row (from r0) of the second segment
  const float beta = a.beta, wgt = a.one_minus_beta / (float)NR;
  FewWarp &fw = fw_all[warp];

  for (int q = tid; q < kSegsPerCta * kFewWarps * kFewSets; q += kFewThreads) {
    (&fs.flips[0][0][0])[q] = 0u;
    (&fs.bits[0][0][0])[q] = 0u;
  }
  if (tid < kSegsPerCta * kFewWarps) (&fs.m_varies[0][0])[tid] = 0u;
  if (tid == 0) fs.timed_out = 0;
  for (int q = lane; q < kSegsPerCta * (kFewSets * 4 + 2); q += 32) (&fw.acc[0][0])[q] = 0.;
  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < kStageDepth; ++st) mbar_init(smem_addr(&fw.bar[st]), 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();                                           // fs.ptr is in place, the barriers are ready
  if (tid < kSegsPerCta * NR) {
    const int sg = tid / NR, r = tid - sg * NR;
    const size_t sample_off = (size_t)(b0 + sg) * a.T * a.d;
    if (sg == 0 || cut < r1) fs.x0[sg][r] = fs.ptr[r][sample_off];
  } else if (tid >= 32 && tid < 32 + kSegsPerCta) {
    const int sg = tid - 32;
    if (sg == 0 || cut < r1) fs.m0bits[sg] = __float_as_uint(load_m1<kBf16>(m_in, (size_t)(b0 + sg) * a.T * a.d));
  }

  // the warp's tiles: tile number j = warp + t * kFewWarps is row r0 + j / tiles_per_row, 512
  // columns from (j % tiles_per_row) * 512 on; stage t % kStageDepth holds it.  The producer runs
  // kStageDepth tiles ahead of the consumer.  (Row and column are worked out from j each time:
  // a division per tile costs less than the registers a running cursor would hold.)
  auto issue = [&](int pt) {                                 // fills stage pt % kStageDepth with the warp's tile pt
    const int pj = warp + pt * kFewWarps;
    if (pj < n_tiles && lane == 0) {
      const int p_rr = pj / tiles_per_row, p_seg = pj - p_rr * tiles_per_row;
      const int st = pt % kStageDepth;
      const size_t off = (size_t)(r0 + p_rr) * a.d + (size_t)p_seg * (32 * kUnroll * 8);
      int vc = 32 * kUnroll;                                 // chunks of this tile that exist
      if (!kFull && chunks - p_seg * 32 * kUnroll < vc) vc = chunks - p_seg * 32 * kUnroll;
      const unsigned bar = smem_addr(&fw.bar[st]), dst = smem_addr(&fw.stage[st][0]);
      if (SENTINEL_BOUNDS(kSiteStageRef, off, (long long)vc * 8, a.ref_extent) &&
          SENTINEL_BOUNDS(kSiteStageX, off, (long long)vc * 8, a.x_extent)) {
        mbar_arrive_expect(bar, (unsigned)vc * (kRefChunkBytes + 16u * NR));
        bulk_copy_in(dst, static_cast<const unsigned char *>(m_in) + off * (kBf16 ? 2 : 4), (unsigned)vc * kRefChunkBytes, bar);
#pragma unroll
        for (int r = 0; r < NR; ++r)
          bulk_copy_in(dst + kTileBytesM + r * kTileBytesX, fs.ptr[r] + off, (unsigned)vc * 16u, bar);
      } else {
        mbar_arrive_expect(bar, 0u);                         // (checked build: nothing is copied, the wait still ends)
      }
    }
  };
#pragma unroll
  for (int st = 0; st < kStageDepth; ++st) issue(st);
  __syncthreads();                                           // fs.x0, fs.m0bits

  float sx[NR], sxx[NR], sxm[NR], ab[NR], x0f[NR];
  unsigned fl[NR], xd[NR];
  unsigned m_diff = 0u;
  float g_sm = 0.f, g_smm = 0.f;
#pragma unroll
  for (int r = 0; r < NR; ++r) { sx[r] = sxx[r] = sxm[r] = ab[r] = 0.f; fl[r] = xd[r] = 0u; }
  int sg = 0;                                                // the segment this warp is in
  auto enter_segment = [&]() {                               // the shift values of segment sg
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      x0f[r] = __uint_as_float(fs.x0[sg][r] << 16);
    }
  };
  enter_segment();
  auto fold = [&]() {                                        // the short fp32 runs: lanes added up, into the warp's fp64 sums
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const float v0 = warp_sum(sx[r]), v1 = warp_sum(sxx[r]), v2 = warp_sum(sxm[r]), v3 = warp_sum(ab[r]);
      if (lane == 0) {
        fw.acc[sg][r * 4 + 0] += (double)v0;
        fw.acc[sg][r * 4 + 1] += (double)v1;
        fw.acc[sg][r * 4 + 2] += (double)v2;
        fw.acc[sg][r * 4 + 3] += (double)v3;
      }
      sx[r] = sxx[r] = sxm[r] = ab[r] = 0.f;
    }
    const float v4 = warp_sum(g_sm), v5 = warp_sum(g_smm);
    if (lane == 0) {
      fw.acc[sg][NR * 4 + 0] += (double)v4;
      fw.acc[sg][NR * 4 + 1] += (double)v5;
    }
    g_sm = g_smm = 0.f;
  };
  auto leave_segment = [&]() {                               // counts and bits of segment sg, per warp
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const unsigned wf = __reduce_add_sync(0xffffffffu, fl[r]);
      const unsigned wx = __reduce_or_sync(0xffffffffu, xd[r]);
      if (lane == 0) {
        fs.flips[sg][warp][r] = wf / kFlipUnit;
        if (wx) atomicOr(&fs.bits[sg][warp][r], (unsigned)kBitXVaries);   // (the non-finite bit may be there already)
      }
      fl[r] = xd[r] = 0u;
    }
    const unsigned wm = __reduce_or_sync(0xffffffffu, m_diff);
    if (lane == 0) fs.m_varies[sg][warp] = wm;
    m_diff = 0u;
  };

  int t = 0;
  unsigned m0bits = fs.m0bits[0];
  float m0 = __uint_as_float(m0bits);
  bool alive = true;
  for (int j = warp; j < n_tiles; j += kFewWarps, ++t) {
    const int rr = j / tiles_per_row, seg = j - rr * tiles_per_row;
    if (sg == 0 && rr >= cut_rr) {                           // this warp enters the second segment
      fold();
      leave_segment();
      sg = 1;
      m0bits = fs.m0bits[1];
      m0 = __uint_as_float(m0bits);
      enter_segment();
    }
    const int st = t % kStageDepth;
    if (!__all_sync(0xffffffffu, mbar_wait(smem_addr(&fw.bar[st]), (unsigned)(t / kStageDepth) & 1u))) {
      alive = false;                                         // the tile never arrived: give up on this warp's rows
      break;
    }
    const size_t off = (size_t)(r0 + rr) * a.d;
    const int base = seg * 32 * kUnroll;
    const unsigned char *stage = fw.stage[st];
    // chunk by chunk: the chunk of m, every tensor's chunk against it, the candidate's chunk out
    unsigned zmin = 0x7F7F7F7Fu;                             // smallest magnitudes met in the tensors' tiles
    unsigned fast_chunks = 0u;                               // chunks that took the packed sign test
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const bool ok = kFull || (base + u * 32 + lane < chunks);
      F8 mv;
      unsigned msp[4];
      float sum[8];
      float mmin = 1.f;
      if (ok) {
        if (kBf16) {
          mv = widen_bf16x8(*reinterpret_cast<const uint4 *>(stage + (size_t)(u * 32 + lane) * 16));
        } else {
          const float4 *src = reinterpret_cast<const float4 *>(stage + (size_t)(u * 32 + lane) * 32);
          const float4 lo = src[0], hi = src[1];
          mv.v[0] = lo.x; mv.v[1] = lo.y; mv.v[2] = lo.z; mv.v[3] = lo.w;
          mv.v[4] = hi.x; mv.v[5] = hi.y; mv.v[6] = hi.z; mv.v[7] = hi.w;
        }
        mmin = fminf(fminf(fminf(fabsf(mv.v[0]), fabsf(mv.v[1])), fminf(fabsf(mv.v[2]), fabsf(mv.v[3]))),
                     fminf(fminf(fabsf(mv.v[4]), fabsf(mv.v[5])), fminf(fabsf(mv.v[6]), fabsf(mv.v[7]))));
#pragma unroll
        for (int e = 0; e < 8; ++e) {                        // the reference's own sums, once per tile
          sum[e] = 0.f;
          const float ms = mv.v[e] - m0;
          g_sm += ms;
          g_smm = fmaf(ms, ms, g_smm);
          m_diff |= __float_as_uint(mv.v[e]) ^ m0bits;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)                          // byte 3 of each m of a pair into bytes 1 and 3
          msp[q] = __byte_perm(__float_as_uint(mv.v[2 * q]), __float_as_uint(mv.v[2 * q + 1]), 0x7733);
      }
      // an exact zero in this chunk of m (for any lane): the general sign test serves
      const bool any_zero = __any_sync(0xffffffffu, !(mmin > 0.f));
      if (!any_zero) fast_chunks |= 1u << u;
      if (ok) {
#pragma unroll
        for (int r = 0; r < NR; ++r) {                       // the tensors, in order
          const uint4 cur = *reinterpret_cast<const uint4 *>(stage + kTileBytesM + r * kTileBytesX + (size_t)(u * 32 + lane) * 16);
          const unsigned x0pair = __byte_perm(__float_as_uint(x0f[r]), 0u, 0x3232);   // the bf16 pattern in both halves
          if (any_zero) few_chunk<true>(cur, mv, msp, x0f[r], m0, x0pair, sum, sx[r], sxx[r], sxm[r], ab[r], fl[r], xd[r], zmin);
          else few_chunk<false>(cur, mv, msp, x0f[r], m0, x0pair, sum, sx[r], sxx[r], sxm[r], ab[r], fl[r], xd[r], zmin);
        }
        // Eq. 1 with the mean over the tensors
#pragma unroll
        for (int e = 0; e < 8; ++e) mv.v[e] = fmaf(beta, mv.v[e], wgt * sum[e]);
        if (SENTINEL_BOUNDS(kSiteRefOut, off + (size_t)(base + u * 32 + lane) * 8, 8, a.ref_extent))
          store_m8<kBf16>(m_out, off + (size_t)(base + u * 32 + lane) * 8, mv);
      }
    }
    unsigned valid = 0u;                                     // this lane's chunks of the tile
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (kFull || base + u * 32 + lane < chunks) valid |= 1u << u;
    // a tile with an exact zero in some tensor: where the packed test ran, a zero whose sign bit
    // equals that of m was not counted
    if (__any_sync(0xffffffffu, ((zmin & 0x7FFFu) == 0u) || ((zmin & 0x7FFF0000u) == 0u))) {
#pragma unroll
      for (int r = 0; r < NR; ++r) fl[r] += kFlipUnit * few_uncounted_zeros(stage, r, lane, valid & fast_chunks, kBf16 ? 1 : 0);
    }
    // a sum of |x - m| that is not a finite number: look at the exponent bits of that tensor's tile
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      if (__any_sync(0xffffffffu, !(ab[r] <= 3.4028234664e38f))) {
        if (few_nonfinite_in_tile(stage, r, lane, valid)) atomicOr(&fs.bits[sg][warp][r], (unsigned)kBitNonfinite);
      }
    }
    // every lane has used what it read from the stage (the sums above depend on it): refill it
    __syncwarp();
    issue(t + kStageDepth);
    if ((t & (kFoldTiles - 1)) == kFoldTiles - 1) fold();
  }
  if (!alive) {
    // the copies still in flight target this CTA's shared memory: give them the same time to land
    for (int k = 1; k < kStageDepth; ++k) {
      const int tt = t + k;
      if (warp + tt * kFewWarps < n_tiles) mbar_wait(smem_addr(&fw.bar[tt % kStageDepth]), (unsigned)(tt / kStageDepth) & 1u);
    }
    if (lane == 0) fs.timed_out = 1;
  }
  fold();
  leave_segment();

  // warps -> CTA in a fixed order
  __syncthreads();
  if (tid == 0 && fs.timed_out) atomicExch(&a.hs->error, kErrStagingTimeout);
  if (tid < kSegsPerCta * NR * kSlotWords) {
    const int sgm = tid / (NR * kSlotWords), r = (tid / kSlotWords) % NR, w8 = tid % kSlotWords;
    unsigned long long *slot = partials + (((size_t)fs.widx[r] * a.G + c) * kSegsPerCta + sgm) * kSlotWords;
    if (!SENTINEL_BOUNDS(kSiteSlot, (((size_t)fs.widx[r] * a.G + c) * kSegsPerCta + sgm) * kSlotWords, kSlotWords, a.partials_words)) {
      // (checked build: the slot lies outside the buffer; nothing is written)
    } else if (sgm == 1 && cut >= r1) {
      if (w8 == 7) slot[7] = 0ull;                           // no second segment: tag 0, unused
    } else {
      unsigned long long out;
      if (w8 < 6) {
        const int q = (w8 == 0) ? r * 4 + 0 : (w8 == 1) ? r * 4 + 1 : (w8 == 2) ? NR * 4 + 0
                    : (w8 == 3) ? NR * 4 + 1 : (w8 == 4) ? r * 4 + 2 : r * 4 + 3;
        double v = 0.;
        for (int w = 0; w < kFewWarps; ++w) v += fw_all[w].acc[sgm][q];
        out = (unsigned long long)__double_as_longlong(v);
      } else if (w8 == 6) {
        out = 0ull;
        for (int w = 0; w < kFewWarps; ++w) out += fs.flips[sgm][w][r];
      } else {
        out = ((unsigned long long)(b0 + sgm + 1) << kTagShift) | ((unsigned long long)fs.x0[sgm][r] << kX0Shift) |
              ((unsigned long long)fs.m0bits[sgm] << kM0Shift);
        for (int w = 0; w < kFewWarps; ++w) out |= fs.bits[sgm][w][r] | (fs.m_varies[sgm][w] ? kBitMVaries : 0ull);
      }
      slot[w8] = out;
    }
  }
}

template <bool kBf16>
__device__ __forceinline__ void few_dispatch(int n, const StreamArgs &a, unsigned long long *partials, int b0,
                                             long long r0, long long cut, long long r1, const void *m_in, void *m_out,
                                             int c, FewShared &fs, double *s_dyn) {
  FewWarp *fw = reinterpret_cast<FewWarp *>(s_dyn);
  if (a.d % (32 * kUnroll * 8) == 0) {
    switch (n) {
      case 1: few_rows<1, true, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      case 2: few_rows<2, true, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      case 3: few_rows<3, true, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      default: few_rows<4, true, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
    }
  } else {
    switch (n) {
      case 1: few_rows<1, false, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      case 2: few_rows<2, false, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      case 3: few_rows<3, false, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
      default: few_rows<4, false, kBf16>(a, partials, b0, r0, cut, r1, m_in, m_out, c, fs, fw); break;
    }
  }
}

// (n_sets tensors share the tile of m: the R workers of a stage, or the B samples of one tensor
// when the reference is a single [T,d] tensor for all of them)
template <bool kBf16>
__device__ void replica_segment(const ReplicaArgs &ra, int n_sets, int b, long long row_a, long long row_b,
                                const void *m_in, void *m_out, unsigned streamed, int c, int sgm,
                                ReplicaShared &sh) {
  const StreamArgs &a = ra.s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = a.d >> 3;                               // d is a multiple of 8 here
  const int tiles_per_row = (chunks + 32 * kUnroll - 1) / (32 * kUnroll);
  const int n_tiles = (int)(row_b - row_a) * tiles_per_row;
  const size_t sample_off = (size_t)b * a.T * a.d;
  const float beta = a.beta, wgt = a.one_minus_beta / (float)__popc(streamed);

  __syncthreads();                                           // the previous segment is done with sh
  for (int i = threadIdx.x; i < kWarps * kMaxWorkers; i += kThreads) {
    const int w = i / kMaxWorkers, r = i - w * kMaxWorkers;
    sh.acc[w][r][0] = sh.acc[w][r][1] = sh.acc[w][r][2] = sh.acc[w][r][3] = 0.;
    sh.flips[w][r] = 0ull;
    sh.bits[w][r] = 0u;
  }
  if (threadIdx.x < kWarps) { sh.m_acc[threadIdx.x][0] = sh.m_acc[threadIdx.x][1] = 0.; sh.m_varies[threadIdx.x] = 0u; }
  if (threadIdx.x < n_sets && ((streamed >> threadIdx.x) & 1u)) sh.x0[threadIdx.x] = ra.xs[threadIdx.x][sample_off];
  const unsigned m0bits = __float_as_uint(load_m1<kBf16>(m_in, sample_off));
  const float m0 = __uint_as_float(m0bits);
  __syncthreads();

  const int first = __ffs(streamed) - 1;
  const int step_rr = kWarps / tiles_per_row, step_seg = kWarps % tiles_per_row;
  int rr = warp / tiles_per_row, seg = warp % tiles_per_row;
  for (int j = warp; j < n_tiles; j += kWarps) {
    const size_t off = (size_t)(row_a + rr) * a.d;
    const int base = seg * 32 * kUnroll;
    F8 mv[kUnroll];
    uint4 xv[kUnroll];
    bool ok[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int ch = base + u * 32 + lane;
      ok[u] = ch < chunks;
      if (ok[u]) {
        mv[u] = load_m8<kBf16>(m_in, off + (size_t)ch * 8);
        xv[u] = ld_x128(ra.xs[first] + off + (size_t)ch * 8);
      }
    }
    // the reference's own sums, once per tile
    float g_sm = 0.f, g_smm = 0.f;
    unsigned m_diff = 0u;
    bool zero_in_m = false;
    float sum[kUnroll][8];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        sum[u][e] = 0.f;
        if (ok[u]) {
          const float ms = mv[u].v[e] - m0;
          g_sm += ms;
          g_smm = fmaf(ms, ms, g_smm);
          m_diff |= __float_as_uint(mv[u].v[e]) ^ m0bits;
          zero_in_m |= (mv[u].v[e] == 0.f);
        }
      }
    }
    const bool any_zero = __any_sync(0xffffffffu, zero_in_m);

    for (unsigned rem = streamed; rem != 0u;) {              // the workers, in order
      const int r = __ffs(rem) - 1;
      rem &= rem - 1u;
      uint4 cur[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) cur[u] = xv[u];
      if (rem != 0u) {                                       // the next worker's tile, ahead of the arithmetic
        const uint16_t *xn = ra.xs[__ffs(rem) - 1] + off;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
          if (ok[u]) xv[u] = ld_x128(xn + (size_t)(base + u * 32 + lane) * 8);
      }
      const unsigned x0 = sh.x0[r], x0pair = x0 | (x0 << 16);
      const float x0f = __uint_as_float(x0 << 16);
      float sx = 0.f, sxx = 0.f, sxm = 0.f, ab = 0.f;
      unsigned flips = 0u, nf = 0u, x_diff = 0u;
      if (any_zero) replica_tile<true>(cur, mv, ok, x0f, m0, x0pair, sum, sx, sxx, sxm, ab, flips, nf, x_diff);
      else replica_tile<false>(cur, mv, ok, x0f, m0, x0pair, sum, sx, sxx, sxm, ab, flips, nf, x_diff);
      sx = warp_sum(sx); sxx = warp_sum(sxx); sxm = warp_sum(sxm); ab = warp_sum(ab);
      flips = __reduce_add_sync(0xffffffffu, flips);
      nf = __reduce_or_sync(0xffffffffu, nf);
      x_diff = __reduce_or_sync(0xffffffffu, x_diff);
      if (lane == 0) {
        sh.acc[warp][r][0] += (double)sx;
        sh.acc[warp][r][1] += (double)sxx;
        sh.acc[warp][r][2] += (double)sxm;
        sh.acc[warp][r][3] += (double)ab;
        sh.flips[warp][r] += flips;
        sh.bits[warp][r] |= (nf ? (unsigned)kBitNonfinite : 0u) | (x_diff ? (unsigned)kBitXVaries : 0u);
      }
    }
    g_sm = warp_sum(g_sm);
    g_smm = warp_sum(g_smm);
    m_diff = __reduce_or_sync(0xffffffffu, m_diff);
    if (lane == 0) {
      sh.m_acc[warp][0] += (double)g_sm;
      sh.m_acc[warp][1] += (double)g_smm;
      sh.m_varies[warp] |= m_diff;
    }
    // Eq. 1 with the mean over the collected workers, written where ema_mean_kernel would put it
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (!ok[u]) continue;
#pragma unroll
      for (int e = 0; e < 8; ++e) mv[u].v[e] = fmaf(beta, mv[u].v[e], wgt * sum[u][e]);
      store_m8<kBf16>(m_out, off + (size_t)(base + u * 32 + lane) * 8, mv[u]);
    }
    rr += step_rr;
    seg += step_seg;
    if (seg >= tiles_per_row) { seg -= tiles_per_row; ++rr; }
  }

  __syncthreads();
  // warps -> CTA in a fixed order, one thread per (worker, slot word)
  if (threadIdx.x < n_sets * kSlotWords) {
    const int r = threadIdx.x / kSlotWords, w8 = threadIdx.x - r * kSlotWords;
    if ((streamed >> r) & 1u) {
      unsigned long long out;
      if (w8 < 6) {
        double t = 0.;
        for (int w = 0; w < kWarps; ++w)
          t += (w8 == 0) ? sh.acc[w][r][0] : (w8 == 1) ? sh.acc[w][r][1] : (w8 == 2) ? sh.m_acc[w][0]
             : (w8 == 3) ? sh.m_acc[w][1] : (w8 == 4) ? sh.acc[w][r][2] : sh.acc[w][r][3];
        out = (unsigned long long)__double_as_longlong(t);
      } else if (w8 == 6) {
        out = 0ull;
        for (int w = 0; w < kWarps; ++w) out += sh.flips[w][r];
      } else {
        out = ((unsigned long long)(b + 1) << kTagShift) | ((unsigned long long)sh.x0[r] << kX0Shift) |
              ((unsigned long long)m0bits << kM0Shift);
        for (int w = 0; w < kWarps; ++w) out |= sh.bits[w][r] | (sh.m_varies[w] ? kBitMVaries : 0ull);
      }
      ra.partials[(((size_t)r * a.G + c) * kSegsPerCta + sgm) * kSlotWords + w8] = out;
    }
  }
}

// (kFew: a handle that follows at most kFewSets workers -- their sums stay in registers; a kernel
// of its own, with its own CTA size, so that neither form pays for the other's registers)
template <bool kFew, bool kBf16 = false>
__global__ void __launch_bounds__(kFew ? kFewThreads : kThreads)
replica_kernel(const ReplicaArgs ra) {
  __shared__ typename std::conditional<kFew, FewShared, ReplicaShared>::type sh;
  __shared__ int s_last;
  extern __shared__ __align__(128) double s_dyn[];   // CTA 0: the refresh's working copies; the others: the warps' staging rings
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const StreamArgs &a = ra.s;
  const bool warmup = (a.mode == kModeReplicaWarmup);
  const int act = __ldcg(&a.hs->kind[a.kind].active);
  // collected: everybody in the warm-up; afterwards whoever is neither banned nor tainted at
  // another stage (both known before the launch: bans only change in the last CTA)
  unsigned streamed = 0u;
  for (int r = 0; r < a.R; ++r) {
    const bool skip = !warmup && (__ldcg(&a.hs->banned[r]) != 0 || ((ra.tainted_in >> r) & 1u));
    if (!skip) streamed |= 1u << r;
  }

  if (blockIdx.x == 0) {
    KindState *ks = &a.hs->kind[a.kind];
    if (ks->refresh_pending)
      refresh_thresholds(ks, a.hist, a.sorted, a.cap0, a.cap1, a.units0, a.units1, a.n_metrics, a.a5, s_dyn);
  } else if (streamed != 0u) {
    const int c = blockIdx.x - 1;
    const long long rows = (long long)a.B * a.T;
    const long long r0 = (rows * c) / a.G, r1 = (rows * (c + 1)) / a.G;
    const int n_streamed = __popc(streamed);
    if constexpr (kFew) {
      if (threadIdx.x == 0) {                                // the tensors that stream, in worker order
        int n = 0;
        for (int r = 0; r < a.R; ++r)
          if ((streamed >> r) & 1u) { sh.ptr[n] = ra.xs[r]; sh.widx[n] = r; ++n; }
      }
    }
    // segment 0: the CTA's rows up to the end of the sample its first row lies in; segment 1: the
    // rest, if any
    const int b0 = (int)(r0 / a.T);
    const long long cut = ((long long)(b0 + 1) * a.T < r1) ? (long long)(b0 + 1) * a.T : r1;
    if constexpr (kFew) {
      few_dispatch<kBf16>(n_streamed, a, ra.partials, b0, r0, cut, r1, a.ema[act], a.ema[act ^ 1], c, sh, s_dyn);
    } else {
      for (int sgm = 0; sgm < kSegsPerCta; ++sgm) {
        const long long row = sgm ? cut : r0, row_b = sgm ? r1 : cut;
        if (row < row_b)
          replica_segment<kBf16>(ra, a.R, b0 + sgm, row, row_b, a.ema[act], a.ema[act ^ 1], streamed, c, sgm, sh);
        else if (threadIdx.x < a.R)
          ra.partials[(((size_t)threadIdx.x * a.G + c) * kSegsPerCta + sgm) * kSlotWords + 7] = 0ull;   // unused
      }
    }
  }

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned t = atomicAdd(a.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // the worker loop: scores, test, counters, history, one worker after the other
  const int rows = a.B + 1;
  for (int r = 0; r < a.R; ++r) {
    const FinalizeTarget ft = {r, ra.partials + (size_t)r * a.G * kSegsPerCta * kSlotWords,
                               ra.scores_all + (size_t)r * rows * a.n_metrics,
                               ra.flags_all ? ra.flags_all + (size_t)r * rows : nullptr,
                               ra.sw_all ? ra.sw_all + (size_t)r * rows : nullptr,
                               (!warmup && ((ra.tainted_in >> r) & 1u)) ? 1 : 0, r == a.R - 1, 0};
    finalize(a, ft);
    __threadfence();                           // the next pass reads the state this one wrote
    __syncthreads();
  }
  // nobody flagged: the mean over all collected workers is already in the spare buffer
  if (threadIdx.x == 0) {
    KindState *ks = &a.hs->kind[a.kind];
    const unsigned collected = __ldcg(&ks->step_collected), tainted = __ldcg(&ks->step_tainted);
    if (collected != 0u && tainted == 0u) {
      ks->active = act ^ 1;
      ks->mean_done_step = __ldcg(&ks->steps);
    }
  }
}

// One [T,d] reference for all B samples of a tensor (a variant the paper does not state: the
// reference of Eq. 1 follows the mean over the samples).  The streaming side is the multi-worker
// one with the samples in the workers' place -- a tile of m against the B samples' tiles, the
// candidate m' = beta m + (1-beta)/B sum_b x[b] into the spare buffer -- over the T token rows;
// the last CTA then finalizes as for any single submission (every sample a unit, all or nothing
// commit).  2 + 8/B bytes per element of x.
// (kFew: at most kFewSets samples, as for the workers above)
template <bool kFew>
__global__ void __launch_bounds__(kFew ? kFewThreads : kThreads)
shared_ref_kernel(const ReplicaArgs ra) {
  __shared__ typename std::conditional<kFew, FewShared, ReplicaShared>::type sh;
  __shared__ int s_last;
  extern __shared__ __align__(128) double s_dyn[];
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const StreamArgs &a = ra.s;
  const int act = __ldcg(&a.hs->kind[a.kind].active);
  const unsigned all = (a.B >= 32) ? 0xffffffffu : ((1u << a.B) - 1u);
  if (blockIdx.x == 0) {
    KindState *ks = &a.hs->kind[a.kind];
    if (ks->refresh_pending)
      refresh_thresholds(ks, a.hist, a.sorted, a.cap0, a.cap1, a.units0, a.units1, a.n_metrics, a.a5, s_dyn);
  } else {
    const int c = blockIdx.x - 1;
    const long long r0 = ((long long)a.T * c) / a.G, r1 = ((long long)a.T * (c + 1)) / a.G;   // token rows
    if constexpr (kFew) {
      if (threadIdx.x < a.B) { sh.ptr[threadIdx.x] = ra.xs[threadIdx.x]; sh.widx[threadIdx.x] = threadIdx.x; }
      few_dispatch<false>(a.B, a, ra.partials, 0, r0, r1, r1, a.ema[act], a.ema[act ^ 1], c, sh, s_dyn);
    } else {
      replica_segment<false>(ra, a.B, 0, r0, r1, a.ema[act], a.ema[act ^ 1], all, c, 0, sh);
    }
    if (!kFew && threadIdx.x < a.B)              // the second slot of every pair stays unused
      ra.partials[(((size_t)threadIdx.x * a.G + c) * kSegsPerCta + 1) * kSlotWords + 7] = 0ull;
  }

  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned t = atomicAdd(a.ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const FinalizeTarget ft = {0, ra.partials, a.scores_out, a.flags_out, nullptr, 0, 1, 1};
  finalize(a, ft);
}

// Brings both kinds' thresholds up to date outside a streaming launch (queries, export).
__global__ void __launch_bounds__(kThreads)
refresh_kernel(HandleState *hs, double *hist_act, double *hist_grad, double *sorted_act,
               double *sorted_grad, int cap0, int cap1, int units0, int units1, int n_metrics,
               Alg5Params a5_act, Alg5Params a5_grad) {
  extern __shared__ double s_dyn[];
  if (hs->kind[0].refresh_pending)
    refresh_thresholds(&hs->kind[0], hist_act, sorted_act, cap0, cap1, units0, units1, n_metrics, a5_act, s_dyn);
  __syncthreads();
  if (hs->kind[1].refresh_pending)
    refresh_thresholds(&hs->kind[1], hist_grad, sorted_grad, cap0, cap1, units0, units1, n_metrics, a5_grad, s_dyn);
}

// Alg. 4 (GradientReplacement) for the one submission a handle sees: if the last verified step
// of this kind was flagged, the outgoing tensor is overwritten with the reference m_{t-1}
// rounded to bf16 (or with zeros, the variant of the SWARM appendix); otherwise nothing is
// touched.  The decision is read on the device, so the call needs no host round trip.  A
// flagged step did not commit, so the active buffer still holds m_{t-1}.
// Traffic when it replaces: 4 B read + 2 B written per element (2 B written when zero-filling).
constexpr int kReplaceThreads = 256;

__device__ __forceinline__ void st_x128(uint16_t *p, const uint4 &v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__global__ void __launch_bounds__(kReplaceThreads)
replace_kernel(const HandleState *hs, int kind, const void *ema0, const void *ema1, int ema_bf16, uint16_t *x,
               long long n_chunks, long long ref_chunks, long long sample_chunks, int zero_fill,
               unsigned *replaced_out) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const KindState *ks = &hs->kind[kind];
  const int flagged = ks->last_flagged;
  if (blockIdx.x == 0 && threadIdx.x == 0 && replaced_out) *replaced_out = flagged ? 1u : 0u;
  if (!flagged) return;
  const void *m = ks->active ? ema1 : ema0;
  const long long stride = (long long)gridDim.x * kReplaceThreads;
  for (long long c = (long long)blockIdx.x * kReplaceThreads + threadIdx.x; c < n_chunks; c += stride) {
    uint4 out = make_uint4(0u, 0u, 0u, 0u);
    // a [T,d] or [d] reference repeats every ref_chunks; a [B,d] one holds a row of ref_chunks per sample
    const long long cm = sample_chunks ? (c / sample_chunks) * ref_chunks + c % ref_chunks
                                       : ref_chunks ? c % ref_chunks : c;
    if (!SENTINEL_BOUNDS(kSiteReplace, c, 1, n_chunks) ||
        !SENTINEL_BOUNDS(kSiteReplace, cm, 1, sample_chunks ? (n_chunks / sample_chunks) * ref_chunks : ref_chunks ? ref_chunks : n_chunks))
      continue;
    if (!zero_fill && ema_bf16) {                 // the reference already is a bf16 tensor
      out = ld_x128(static_cast<const uint16_t *>(m) + cm * 8);
    } else if (!zero_fill) {
      const F8 v = ld_m256(static_cast<const float *>(m) + cm * 8);
      out.x = pack_bf16x2_rn(v.v[0], v.v[1]);
      out.y = pack_bf16x2_rn(v.v[2], v.v[3]);
      out.z = pack_bf16x2_rn(v.v[4], v.v[5]);
      out.w = pack_bf16x2_rn(v.v[6], v.v[7]);
    }
    st_x128(x + c * 8, out);
  }
}

// Second half of a multi-worker iteration (Alg. 1 main loop, Eq. 1): after every worker has
// been scored, decide who is tainted -- the flagged workers and, for gradients (Alg. 3), the
// ones tainted at another stage, unless more than half of the workers still in the pool are in
// that set, which Alg. 2 / Alg. 3 read as a natural distribution shift and clear -- and move the
// reference with the mean over the clean collected workers, in place:
//   m <- beta m + (1 - beta) / |clean| * sum_{r clean} x^(r).
// When nobody was flagged the scoring launch has already put that mean in place (it marks the
// iteration in mean_done_step) and only the report bits are left to do here.
// Every CTA derives the same clean set from the masks the scoring launch left in the state.
// Traffic when it runs: 4 B read + 4 B written of m and 2 B per clean worker, per element.
struct WorkerPointers { const uint16_t *x[kMaxWorkers]; };

template <bool kBf16>
__global__ void __launch_bounds__(kReplaceThreads)
ema_mean_kernel(HandleState *hs, int kind, WorkerPointers xs, void *ema0, void *ema1, long long n_chunks,
                int R, int rows, float beta, float one_minus_beta, int warmup, unsigned *flags_out) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  KindState *ks = &hs->kind[kind];
  const unsigned collected = ks->step_collected, tainted = ks->step_tainted, nonfinite = ks->step_nonfinite;
  int n_banned = 0;
  for (int r = 0; r < R; ++r) n_banned += hs->banned[r] != 0;
  const int n_stage = __popc(tainted) + (kind == 1 ? __popc(ks->step_elsewhere) : 0);   // the stage's tainted set
  const bool natural = !warmup && 2 * n_stage > R - n_banned;
  const unsigned clean = collected & ~(natural ? nonfinite : tainted);
  const int n_clean = __popc(clean);
  const bool done = ks->mean_done_step == ks->steps;

  if (blockIdx.x == 0 && threadIdx.x == 0) {
    ks->last_flagged = (n_stage != 0 && !natural) ? 1 : 0;
    if (flags_out)
      for (int r = 0; r < R; ++r)
        flags_out[(size_t)r * rows] |= ((clean >> r) & 1u ? kFlagCommitted : 0u) | (natural ? kFlagNaturalShift : 0u);
  }
  if (n_clean == 0 || done) return;
  void *m = ks->active ? ema1 : ema0;
  const float wgt = one_minus_beta / (float)n_clean;
  const long long stride = (long long)gridDim.x * kReplaceThreads;
  for (long long c = (long long)blockIdx.x * kReplaceThreads + threadIdx.x; c < n_chunks; c += stride) {
    F8 mv = load_m8<kBf16>(m, (size_t)c * 8);
    float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int r = 0; r < R; ++r) {
      if (!((clean >> r) & 1u)) continue;
      const uint4 xv = ld_x128(xs.x[r] + c * 8);
      const unsigned wv[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        sum[2 * j] += __uint_as_float(wv[j] << 16);
        sum[2 * j + 1] += __uint_as_float(wv[j] & 0xFFFF0000u);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) mv.v[j] = fmaf(beta, mv.v[j], wgt * sum[j]);
    store_m8<kBf16>(m, (size_t)c * 8, mv);
  }
}

// The one worker this verifier follows was tainted at another stage in this step: nothing is
// collected or recorded; the step counts and asks for gradient replacement (Alg. 4).
__global__ void skip_tainted_kernel(HandleState *hs, int kind) {
  hs->kind[kind].steps += 1;
  hs->kind[kind].last_flagged = 1;
}

__global__ void reset_worker_kernel(HandleState *hs, int worker) {
  hs->violations[worker] = 0;
  hs->clean_streak[worker] = 0;
  hs->banned[worker] = 0;
}

}  // namespace sentinel
