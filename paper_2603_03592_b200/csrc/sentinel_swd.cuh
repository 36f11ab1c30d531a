// Sliced Wasserstein distance (Sec. 3.1) on the device.  x and m are clouds of tokens in R^d;
// for each of L caller-supplied directions both clouds are projected (a skinny contraction,
// [B*T, d] x [d, L], done while x and m stream through once), the projections of each sample
// are sorted and matched (W1 of two empirical measures = mean |a_(i) - b_(i)|), the samples'
// sorted lists are merged for the whole-tensor unit, and the L terms are averaged.
#pragma once

#include "sentinel_kernels.cuh"

namespace sentinel {

// A projection CTA has 512 or 768 threads; the host takes whichever keeps more threads resident
// per SM (the directions can fill most of the shared memory: then one large CTA is all there is).
constexpr int kSwdSortThreads = 1024;

// Every kernel of the chain is launched with programmatic stream serialization and starts with
// this: the next launch may be set up while this one runs, and nothing is read before the
// previous launch on the stream has completed and flushed (with a plain launch both do nothing).
__device__ __forceinline__ void chain_entry() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
constexpr int kSwdMaxTokensPerSample = 16384;    // one sample's projections are sorted in shared memory

// extents, for the checked build, of what the sort / merge / W1 launches index: floats of one buffer
// of lists (projections, sorted lists, merge buffer: 2L lists of B*T each) and doubles of the per-CTA sums
struct SwdExtents {
  long long list_floats, partial_doubles;
};

// ---------------------------------------------------------------------------------------------
// projections: proj[(t*L + l)*rows + row] = sum_c v[row][c] * u[l][c], t = 0 for x, 1 for m.
// A warp owns whole rows; the directions sit in shared memory as bf16 (they are given as bf16).
// Traffic: x and m are read once, 6 B/element; per element L multiply-adds for each of x and m
// (m is fp32: its half of the work stays on the CUDA cores).
// The reference is m1 if *active is non-zero, else m0 (a verifier keeps two buffers and flips
// between them on the device); every kernel of the chain returns at once if *skip is non-zero
// (a banned worker's tensor is not read).  Both pointers may be nullptr.
//
// Projection is linear and so is Eq. 1: the projections of the reference obey
//   P(m_t) = beta P(m_{t-1}) + (1-beta) P(x_t)
// whenever the reference moves.  A verifier therefore keeps P(m) itself ([rows][L] doubles, two
// buffers pm0 / pm1 selected by the same `active` word as the reference, so a step that does not
// commit leaves them alone).  This kernel computes P(m) from m -- the stateless call, and a
// verifier's first step or its first step after a state import -- and, if the buffers are given,
// stores it in the current one and the candidate P(m_t) in the spare one; from then on
// swd_project_mma_kernel carries the buffers along and reads x only, 2 B/element instead of 6.
// kRefOnly = true projects the reference alone into the current buffer (x is not read, nothing
// else is written): once per iteration of a verifier that follows several workers, whose
// reference moves with the mean over the clean workers rather than by that recursion; its
// workers then all take the x-only launch against the same P(m).
// kBf16: the reference buffers hold bf16 (widened on load; such a verifier projects its reference
// afresh every step, because the rounding of the stored reference does not follow the recursion).
template <int L, int kSwdThreads, bool kRefOnly = false, bool kBf16 = false>
__global__ void __launch_bounds__(kSwdThreads, kSwdThreads == 512 ? 2 : 1)
swd_project_kernel(const uint16_t *x, const void *m0, const void *m1, const int *active, const int *skip,
                   const uint16_t *u, float *proj, long long rows, int d, double *pm0, double *pm1, float beta,
                   float one_minus_beta) {
  extern __shared__ uint4 s_u[];                 // [L][d/8], 8 bf16 each
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const bool second = active && __ldcg(active);
  const void *m = second ? m1 : m0;
  double *pm_cur = second ? pm1 : pm0, *pm_next = second ? pm0 : pm1;
  const int chunks = d >> 3;
  for (int i = threadIdx.x; i < L * chunks; i += kSwdThreads)
    s_u[i] = reinterpret_cast<const uint4 *>(u)[i];
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (kSwdThreads / 32) + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * (kSwdThreads / 32);
  for (long long row = warp; row < rows; row += n_warps) {
    float ax[L], am[L];
#pragma unroll
    for (int l = 0; l < L; ++l) ax[l] = am[l] = 0.f;
    const size_t off = (size_t)row * d;
    // two chunks per trip, their loads issued before any arithmetic (more bytes in flight)
    for (int c0 = lane; c0 < chunks; c0 += 64) {
      uint4 xv[2];
      F8 mv[2];
      bool ok[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = c0 + 32 * h;
        ok[h] = c < chunks;
        if (ok[h]) {
          if (!kRefOnly) xv[h] = ld_x128(x + off + (size_t)c * 8);
          mv[h] = load_m8<kBf16>(m, off + (size_t)c * 8);
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (!ok[h]) continue;
        const int c = c0 + 32 * h;
        float xf[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const unsigned xw = kRefOnly ? 0u : (j == 0 ? xv[h].x : j == 1 ? xv[h].y : j == 2 ? xv[h].z : xv[h].w);
          xf[2 * j] = __uint_as_float(xw << 16);
          xf[2 * j + 1] = __uint_as_float(xw & 0xFFFF0000u);
        }
#pragma unroll
        for (int l = 0; l < L; ++l) {
          const uint4 uv = s_u[l * chunks + c];
          const unsigned uw[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float u_lo = __uint_as_float(uw[j] << 16), u_hi = __uint_as_float(uw[j] & 0xFFFF0000u);
            if (!kRefOnly) {
              ax[l] = fmaf(xf[2 * j], u_lo, ax[l]);
              ax[l] = fmaf(xf[2 * j + 1], u_hi, ax[l]);
            }
            am[l] = fmaf(mv[h].v[2 * j], u_lo, am[l]);
            am[l] = fmaf(mv[h].v[2 * j + 1], u_hi, am[l]);
          }
        }
      }
    }
#pragma unroll
    for (int l = 0; l < L; ++l) {
      const float sx = kRefOnly ? 0.f : warp_sum(ax[l]), sm = warp_sum(am[l]);
      if (lane == l) {
        const size_t at = (size_t)row * L + l;
        if (kRefOnly) {
          pm_cur[at] = (double)sm;
          continue;
        }
        proj[(size_t)l * rows + row] = sx;
        proj[((size_t)L + l) * rows + row] = sm;
        if (pm_cur) {
          pm_cur[at] = (double)sm;
          pm_next[at] = (double)beta * (double)sm + (double)one_minus_beta * (double)sx;
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The incremental projection (x only) on the tensor cores.  [rows, d] x [d, L] with bf16 operands
// is a dense contraction, but a skinny one (L <= 16): it is bound by the one read of x, so what
// matters is that the operands reach the multiplier without a detour.  A warp owns 16 token rows
// and walks along d; lane (g, q) = (lane / 4, lane % 4) fetches with one 128-bit load the 8
// consecutive elements [32*cb + 8*q, +8) of row g and of row g + 8.  Those four words are the A
// fragments of two m16n8k16 multiplies as they stand: a dot product does not care in which order
// its terms are taken, so the multiply's k-slots (2q, 2q+1 | 2q+8, 2q+9) may stand for columns
// (8q, 8q+1 | 8q+2, 8q+3) in the first and (8q+4, 8q+5 | 8q+6, 8q+7) in the second, as long as
// the B fragment -- direction g, same eight columns, one 128-bit load from shared memory --
// pairs them the same way.  Products of bf16 are exact in fp32; the sums are fp32.
// The loads of the next 128 columns are issued before the multiplies of the current ones.
constexpr int kSwdMmaThreads = 512;
constexpr int kSwdMmaWarps = kSwdMmaThreads / 32;

__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                                 unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__host__ __device__ inline int swd_mma_stride(int chunks) {     // uint4 per direction in shared memory, = 4 mod 8:
  return ((chunks + 7) & ~7) + 4;                               // the 8 lanes of a quarter-warp hit 8 different 16-byte banks
}

template <int NB>            // blocks of 8 directions: 1 for L = 4 or 8, 2 for L = 16
__global__ void __launch_bounds__(kSwdMmaThreads, 1)
swd_project_mma_kernel(const uint16_t *x, const int *active, const int *skip, const uint16_t *u, float *proj,
                       long long rows, int d, int L, double *pm0, double *pm1, float beta, float one_minus_beta) {
  extern __shared__ uint4 s_u[];                 // [L][stride], 8 bf16 each
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const bool second = active && __ldcg(active);
  const double *pm_cur = second ? pm1 : pm0;
  double *pm_next = second ? pm0 : pm1;
  const int chunks = d >> 3, stride = swd_mma_stride(chunks);
  for (int i = threadIdx.x; i < L * chunks; i += kSwdMmaThreads) {
    const int l = i / chunks, c = i - l * chunks;
    s_u[l * stride + c] = reinterpret_cast<const uint4 *>(u)[i];
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, q = lane & 3;
  const long long n_tasks = (rows + 15) >> 4;
  const int n_groups = (chunks + 15) >> 4;       // 16 chunks = 128 columns = 4 blocks of 32 per trip
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  // tasks are dealt CTA-first, so that a short list still spreads over all SMs
  for (long long task = blockIdx.x + (long long)gridDim.x * warp; task < n_tasks;
       task += (long long)gridDim.x * kSwdMmaWarps) {
    const long long row_a = task * 16 + g, row_b = row_a + 8;
    // a row past the end is read as the last row and its result dropped (row i of the product
    // depends on row i of x alone)
    const uint16_t *pa = x + (size_t)(row_a < rows ? row_a : rows - 1) * d;
    const uint16_t *pb = x + (size_t)(row_b < rows ? row_b : rows - 1) * d;
    float acc[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;

    uint4 cur[4][2], nxt[4][2];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int c = k * 4 + q;
      cur[k][0] = c < chunks ? ld_x128(pa + (size_t)c * 8) : zero4;
      cur[k][1] = c < chunks ? ld_x128(pb + (size_t)c * 8) : zero4;
    }
    for (int gi = 0; gi < n_groups; ++gi) {
      if (gi + 1 < n_groups) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int c = (gi + 1) * 16 + k * 4 + q;
          nxt[k][0] = c < chunks ? ld_x128(pa + (size_t)c * 8) : zero4;
          nxt[k][1] = c < chunks ? ld_x128(pb + (size_t)c * 8) : zero4;
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = gi * 16 + k * 4 + q;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          const int l = nb * 8 + g;
          const uint4 uv = (l < L && c < chunks) ? s_u[l * stride + c] : zero4;
          mma_bf16_16x8x16(acc[nb], cur[k][0].x, cur[k][1].x, cur[k][0].y, cur[k][1].y, uv.x, uv.y);
          mma_bf16_16x8x16(acc[nb], cur[k][0].z, cur[k][1].z, cur[k][0].w, cur[k][1].w, uv.z, uv.w);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) { cur[k][0] = nxt[k][0]; cur[k][1] = nxt[k][1]; }
    }
    // accumulator layout: [0], [1] = (row g, directions 2q, 2q+1), [2], [3] = (row g + 8, same)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const long long row = (e < 2) ? row_a : row_b;
        const int l = nb * 8 + 2 * q + (e & 1);
        if (row < rows && l < L) {
          const size_t at = (size_t)row * L + l;
          const double p_cur = pm_cur[at];
          const float sx = acc[nb][e];
          proj[(size_t)l * rows + row] = sx;
          proj[((size_t)L + l) * rows + row] = (float)p_cur;
          pm_next[at] = (double)beta * p_cur + (double)one_minus_beta * (double)sx;
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Both projections on the tensor cores: P(x) as above and P(m) of a stored reference.
//
// A bf16 reference is an operand as it stands.  An fp32 one is split, exactly, into three bf16
// terms: hi = the upper 16 bits of m, mid = the upper 16 bits of m - hi, lo = m - hi - mid (a
// 24-bit significand in three pieces of 8; both differences are exact in fp32 and lo needs no
// rounding), so  m . u = hi . u + mid . u + lo . u  with every product exact in fp32 and the three
// multiplies accumulating into the same fp32 sums.  (A reference value that is not finite makes
// the differences, hence the projection, not a number.)
//
// Work is dealt differently from the x-only kernel: a CTA owns 16 token rows at a time and its
// twelve warps split the columns of those rows among them, so every task keeps the whole CTA
// loading (whole-row tasks per warp would leave most warps of an SM without work on the last
// round); the warps' partial sums meet in shared memory and are added in warp order.
constexpr int kSwdRefThreads = 384;
constexpr int kSwdRefWarps = kSwdRefThreads / 32;

template <bool kBf16> struct RefWords;
template <> struct RefWords<true> { uint4 v; };
template <> struct RefWords<false> { F8 v; };

template <bool kBf16>
__device__ __forceinline__ RefWords<kBf16> load_ref8(const void *m, size_t at) {
  RefWords<kBf16> r;
  if constexpr (kBf16) r.v = ld_x128(static_cast<const uint16_t *>(m) + at);
  else r.v = load_m8<false>(m, at);
  return r;
}

// the pair (e, o) as two bf16 in one word (e in the low half), each the upper 16 bits of its float
__device__ __forceinline__ unsigned upper_halves(float e, float o) {
  return __byte_perm(__float_as_uint(e), __float_as_uint(o), 0x7632);
}
__device__ __forceinline__ float upper_part(float v) { return __uint_as_float(__float_as_uint(v) & 0xFFFF0000u); }

// acc += (rows g | g + 8 of the reference, 8 columns) x (direction fragment uv)
template <bool kBf16>
__device__ __forceinline__ void mma_ref8(float (&acc)[4], const RefWords<kBf16> &ra, const RefWords<kBf16> &rb, const uint4 &uv) {
  if constexpr (kBf16) {
    mma_bf16_16x8x16(acc, ra.v.x, rb.v.x, ra.v.y, rb.v.y, uv.x, uv.y);
    mma_bf16_16x8x16(acc, ra.v.z, rb.v.z, ra.v.w, rb.v.w, uv.z, uv.w);
  } else {
    unsigned a[3][4], b[3][4];                    // [term][pair of columns]
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float e = ra.v.v[2 * j], o = ra.v.v[2 * j + 1];
      a[0][j] = upper_halves(e, o);
      e -= upper_part(e); o -= upper_part(o);
      a[1][j] = upper_halves(e, o);
      e -= upper_part(e); o -= upper_part(o);
      a[2][j] = upper_halves(e, o);
      e = rb.v.v[2 * j]; o = rb.v.v[2 * j + 1];
      b[0][j] = upper_halves(e, o);
      e -= upper_part(e); o -= upper_part(o);
      b[1][j] = upper_halves(e, o);
      e -= upper_part(e); o -= upper_part(o);
      b[2][j] = upper_halves(e, o);
    }
#pragma unroll
    for (int t = 2; t >= 0; --t) {                // the small terms first
      mma_bf16_16x8x16(acc, a[t][0], b[t][0], a[t][1], b[t][1], uv.x, uv.y);
      mma_bf16_16x8x16(acc, a[t][2], b[t][2], a[t][3], b[t][3], uv.z, uv.w);
    }
  }
}

template <int NB, bool kWithX, bool kBf16>    // NB blocks of 8 directions; kWithX = false: the reference alone
__global__ void __launch_bounds__(kSwdRefThreads, 1)
swd_project_ref_mma_kernel(const uint16_t *x, const void *m0, const void *m1, const int *active, const int *skip,
                           const uint16_t *u, float *proj, long long rows, int d, int L, double *pm0, double *pm1,
                           float beta, float one_minus_beta) {
  extern __shared__ uint4 s_u[];                 // [L][stride], 8 bf16 each; then the warps' partial sums
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const bool second = active && __ldcg(active);
  const void *m = second ? m1 : m0;
  double *pm_cur = second ? pm1 : pm0, *pm_next = second ? pm0 : pm1;
  const int chunks = d >> 3, stride = swd_mma_stride(chunks);
  constexpr int kSets = kWithX ? 2 : 1, kVals = kSets * NB * 4;     // accumulator words of a lane
  float *s_acc = reinterpret_cast<float *>(s_u + (size_t)L * stride);            // [warp][kVals][32]
  for (int i = threadIdx.x; i < L * chunks; i += kSwdRefThreads) {
    const int l = i / chunks, c = i - l * chunks;
    s_u[l * stride + c] = reinterpret_cast<const uint4 *>(u)[i];
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, q = lane & 3;
  const long long n_tasks = (rows + 15) >> 4;
  const int n_blocks = (chunks + 3) >> 2;        // blocks of 32 columns (4 chunks, one per q)
  const int blk0 = (int)((long long)n_blocks * warp / kSwdRefWarps), blk1 = (int)((long long)n_blocks * (warp + 1) / kSwdRefWarps);
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  RefWords<kBf16> zero_ref;
  if constexpr (kBf16) zero_ref.v = zero4;
  else {
#pragma unroll
    for (int j = 0; j < 8; ++j) zero_ref.v.v[j] = 0.f;
  }
  for (long long task = blockIdx.x; task < n_tasks; task += gridDim.x) {
    const long long row_a = task * 16 + g, row_b = row_a + 8;
    // a row past the end is read as the last row and its result dropped
    const size_t off_a = (size_t)(row_a < rows ? row_a : rows - 1) * d, off_b = (size_t)(row_b < rows ? row_b : rows - 1) * d;
    float acc[kSets][NB][4];
#pragma unroll
    for (int st = 0; st < kSets; ++st)
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) acc[st][nb][0] = acc[st][nb][1] = acc[st][nb][2] = acc[st][nb][3] = 0.f;

    // two blocks of 32 columns per trip; the loads of the next trip are issued before the multiplies of this one
    uint4 xc[2][2], xn[2][2];
    RefWords<kBf16> rc[2][2], rn[2][2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int c = (blk0 + k) * 4 + q;
      const bool ok = blk0 + k < blk1 && c < chunks;
      if constexpr (kWithX) {
        xc[k][0] = ok ? ld_x128(x + off_a + (size_t)c * 8) : zero4;
        xc[k][1] = ok ? ld_x128(x + off_b + (size_t)c * 8) : zero4;
      }
      rc[k][0] = ok ? load_ref8<kBf16>(m, off_a + (size_t)c * 8) : zero_ref;
      rc[k][1] = ok ? load_ref8<kBf16>(m, off_b + (size_t)c * 8) : zero_ref;
    }
    for (int blk = blk0; blk < blk1; blk += 2) {
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int c = (blk + 2 + k) * 4 + q;
        const bool ok = blk + 2 + k < blk1 && c < chunks;
        if constexpr (kWithX) {
          xn[k][0] = ok ? ld_x128(x + off_a + (size_t)c * 8) : zero4;
          xn[k][1] = ok ? ld_x128(x + off_b + (size_t)c * 8) : zero4;
        }
        rn[k][0] = ok ? load_ref8<kBf16>(m, off_a + (size_t)c * 8) : zero_ref;
        rn[k][1] = ok ? load_ref8<kBf16>(m, off_b + (size_t)c * 8) : zero_ref;
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int c = (blk + k) * 4 + q;
        const bool ok = blk + k < blk1 && c < chunks;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          const int l = nb * 8 + g;
          const uint4 uv = (l < L && ok) ? s_u[l * stride + c] : zero4;
          if constexpr (kWithX) {
            mma_bf16_16x8x16(acc[0][nb], xc[k][0].x, xc[k][1].x, xc[k][0].y, xc[k][1].y, uv.x, uv.y);
            mma_bf16_16x8x16(acc[0][nb], xc[k][0].z, xc[k][1].z, xc[k][0].w, xc[k][1].w, uv.z, uv.w);
          }
          mma_ref8<kBf16>(acc[kSets - 1][nb], rc[k][0], rc[k][1], uv);
        }
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        if constexpr (kWithX) { xc[k][0] = xn[k][0]; xc[k][1] = xn[k][1]; }
        rc[k][0] = rn[k][0]; rc[k][1] = rn[k][1];
      }
    }
    // the warps' sums meet in shared memory; the first warps add them in warp order and write
    __syncthreads();                              // (the previous task's sums have been read)
#pragma unroll
    for (int st = 0; st < kSets; ++st)
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) s_acc[(warp * kVals + (st * NB + nb) * 4 + e) * 32 + lane] = acc[st][nb][e];
    __syncthreads();
    // accumulator layout: [0], [1] = (row g, directions 2q, 2q+1), [2], [3] = (row g + 8, same)
    for (int item = threadIdx.x; item < NB * 4 * 32; item += kSwdRefThreads) {
      const int ln = item & 31, e = (item >> 5) & 3, nb = item >> 7;
      const int gg = ln >> 2, qq = ln & 3;
      const long long row = task * 16 + gg + ((e < 2) ? 0 : 8);
      const int l = nb * 8 + 2 * qq + (e & 1);
      if (row >= rows || l >= L) continue;
      float sx = 0.f, sm = 0.f;
      for (int w = 0; w < kSwdRefWarps; ++w) {
        if constexpr (kWithX) sx += s_acc[(w * kVals + nb * 4 + e) * 32 + ln];
        sm += s_acc[(w * kVals + ((kSets - 1) * NB + nb) * 4 + e) * 32 + ln];
      }
      const size_t at = (size_t)row * L + l;
      if constexpr (!kWithX) {
        pm_cur[at] = (double)sm;
      } else {
        proj[(size_t)l * rows + row] = sx;
        proj[((size_t)L + l) * rows + row] = sm;
        if (pm_cur) {
          pm_cur[at] = (double)sm;
          pm_next[at] = (double)beta * (double)sm + (double)one_minus_beta * (double)sx;
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// helpers of the sort / W1 kernels
__device__ __forceinline__ double block_sum_ordered(double v, double *s_red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) s_red[warp] = v;
  __syncthreads();
  double total = 0.;
  if (threadIdx.x == 0)
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += s_red[w];
  return total;                                   // valid in thread 0
}

// One round of the bitonic network on a list in shared memory: every thread takes the 8 entries
// whose indices differ in the three bits sh+2, sh+1, sh, and runs the first `steps` of the
// compare-exchange steps on those bits (highest first) in registers -- three steps of the network
// for one trip through shared memory and one barrier.  k2 is the length of the runs being
// merged: a pair is put in ascending order iff bit k2 of its index is clear.
__device__ __forceinline__ void bitonic_round(float *s_val, int npad, int k2, int sh, int steps) {
  for (int t = threadIdx.x; t < (npad >> 3); t += kSwdSortThreads) {
    const int low = t & ((1 << sh) - 1), base = ((t >> sh) << (sh + 3)) | low;
    float v[8];
    if (sh == 0) {
      const float4 p0 = reinterpret_cast<const float4 *>(s_val + base)[0];
      const float4 p1 = reinterpret_cast<const float4 *>(s_val + base)[1];
      v[0] = p0.x; v[1] = p0.y; v[2] = p0.z; v[3] = p0.w; v[4] = p1.x; v[5] = p1.y; v[6] = p1.z; v[7] = p1.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = s_val[base | (e << sh)];
    }
    const bool up = (base & k2) == 0;
#pragma unroll
    for (int st = 0; st < 3; ++st) {
      if (st < steps) {
        const int bit = 4 >> st;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (!(e & bit)) {
            const float lo = v[e], hi = v[e | bit];
            if ((lo > hi) == up) { v[e] = hi; v[e | bit] = lo; }
          }
        }
      }
    }
    if (sh == 0) {
      reinterpret_cast<float4 *>(s_val + base)[0] = make_float4(v[0], v[1], v[2], v[3]);
      reinterpret_cast<float4 *>(s_val + base)[1] = make_float4(v[4], v[5], v[6], v[7]);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) s_val[base | (e << sh)] = v[e];
    }
  }
  __syncthreads();
}

// one CTA per (sample, direction, cloud) and piece: bitonic sort of a list of projections in shared
// memory (padded with +inf to a power of two, at least 8); the sorted list goes back to global
// memory.  pieces = 1: the sample's T projections; pieces = 2 (T even): each half of them on a CTA of
// its own -- twice the SMs at work where the lists are few -- and a merge round puts the halves
// together.  Also clears the ticket word of swd_w1_kernel, a later launch of the chain.
__global__ void __launch_bounds__(kSwdSortThreads)
swd_sort_samples_kernel(const float *proj, float *sorted, unsigned *ticket, int B, int T_sample, int pieces, int L,
                        long long rows, const int *skip, const SwdExtents ext) {
  extern __shared__ float s_val[];                // [npad]
  chain_entry();
  if (skip && __ldcg(skip)) return;
  if (blockIdx.x == 0 && threadIdx.x == 0) *ticket = 0u;
  const int T = T_sample / pieces;                // entries this CTA sorts
  const int run = blockIdx.x / pieces, piece = blockIdx.x - run * pieces;
  const int list = run / B, b = run - list * B;   // list = cloud * L + direction
  int npad = 8;
  while (npad < T) npad <<= 1;
  const size_t first = (size_t)list * rows + (size_t)b * T_sample + (size_t)piece * T;
  if (!SENTINEL_BOUNDS(kSiteSwdLists, first, T, ext.list_floats)) return;      // (the whole CTA: the list is read and written as one)
  const float *src = proj + first;
  // a projection that is not a number is sorted, merged and matched as +inf: the comparisons and
  // min / max of the later steps then see ordered values only, and the sample's W1 comes out not finite
  for (int i = threadIdx.x; i < npad; i += kSwdSortThreads) {
    const float v = i < T ? src[i] : CUDART_INF_F;
    s_val[i] = v == v ? v : CUDART_INF_F;
  }
  __syncthreads();
  // runs of 2, 4 and 8: all inside a thread's 8 consecutive entries, the direction per pair
  for (int t = threadIdx.x; t < (npad >> 3); t += kSwdSortThreads) {
    float v[8];
    const float4 p0 = reinterpret_cast<const float4 *>(s_val + t * 8)[0];
    const float4 p1 = reinterpret_cast<const float4 *>(s_val + t * 8)[1];
    v[0] = p0.x; v[1] = p0.y; v[2] = p0.z; v[3] = p0.w; v[4] = p1.x; v[5] = p1.y; v[6] = p1.z; v[7] = p1.w;
#pragma unroll
    for (int k2 = 2; k2 <= 8; k2 <<= 1) {
#pragma unroll
      for (int bit = k2 >> 1; bit > 0; bit >>= 1) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (!(e & bit)) {
            const bool up = (((t * 8 + e) & k2) == 0);
            const float lo = v[e], hi = v[e | bit];
            if ((lo > hi) == up) { v[e] = hi; v[e | bit] = lo; }
          }
        }
      }
    }
    reinterpret_cast<float4 *>(s_val + t * 8)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4 *>(s_val + t * 8)[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
  __syncthreads();
  for (int k2 = 16, k = 4; k2 <= npad; k2 <<= 1, ++k) {   // merge runs of k2/2 into runs of k2: steps on bits k-1 .. 0
    int j = k - 1;
    const int head = (j + 1) % 3;                 // a short round first, so that the rest are full ones ending at bit 0
    if (head) { bitonic_round(s_val, npad, k2, j - 2, head); j -= head; }
    for (; j >= 2; j -= 3) bitonic_round(s_val, npad, k2, j - 2, 3);
  }
  float *dst = sorted + first;
  for (int i = threadIdx.x; i < T; i += kSwdSortThreads) dst[i] = s_val[i];
}

// ---------------------------------------------------------------------------------------------
// From the sorted sample lists to W1 of every unit.
//
// A sample: its two lists have T entries each, so W1 = mean_i |a_(i) - b_(i)|.
// The whole tensor: the B sorted runs of a list are merged pairwise, ceil(log2 B) rounds, into one
// sorted list of B*T entries per cloud and direction, and W1 = mean_i |A_(i) - B_(i)| again.
//
// A merge is split the way a merge path is: a thread produces kSwdMergeSpan consecutive entries of
// the output.  One bisection tells it how many entries of the left run come before its first
// output (ties: left run first); its outputs are then among the next kSwdMergeSpan entries of
// either run, which it loads in one go and merges in registers (the smaller halves of a bitonic
// merge network).  Linear work, and one chain of dependent loads per thread instead of one per entry.
//
// The last round does not write its output: a thread merges the same span of the x cloud and of
// the reference cloud and adds up |A_(i) - B_(i)| at once (swd_w1_kernel).  The same launch has
// CTAs for the samples' W1, and the CTA that draws the last ticket adds the per-CTA sums in a
// fixed order and writes the means over the directions: out[0] = the whole tensor, out[1+b] =
// sample b.  The ticket word must be zero at launch (the sort kernel clears it).
constexpr int kSwdMergeSpan = 8;
constexpr int kSwdW1Threads = 256;
constexpr int kSwdW1Span = kSwdW1Threads * kSwdMergeSpan;         // entries a CTA covers

// how many entries of the left run come before merged position d (0 <= d <= la + lb)
__device__ __forceinline__ int merge_split(const float *left, int la, const float *right, int lb, int d) {
  int lo = d > lb ? d - lb : 0, hi = d < la ? d : la;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (left[mid] <= right[d - 1 - mid]) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// merged entries d .. d + 7 of (left, right); +inf past the end
__device__ __forceinline__ void merge_span(const float *left, int la, const float *right, int lb, int d, float (&out)[kSwdMergeSpan]) {
  const int a = merge_split(left, la, right, lb, d), b = d - a;
  float ca[kSwdMergeSpan], cb[kSwdMergeSpan];
#pragma unroll
  for (int k = 0; k < kSwdMergeSpan; ++k) {
    ca[k] = a + k < la ? left[a + k] : CUDART_INF_F;
    cb[k] = b + k < lb ? right[b + k] : CUDART_INF_F;
  }
  // the 8 smallest of two ascending runs of 8: min(ca[k], cb[7-k]) is a bitonic sequence of them
#pragma unroll
  for (int k = 0; k < kSwdMergeSpan; ++k) out[k] = fminf(ca[k], cb[kSwdMergeSpan - 1 - k]);
#pragma unroll
  for (int dist = kSwdMergeSpan / 2; dist > 0; dist >>= 1) {
#pragma unroll
    for (int k = 0; k < kSwdMergeSpan; ++k) {
      if (!(k & dist)) {
        const float lo = fminf(out[k], out[k | dist]), hi = fmaxf(out[k], out[k | dist]);
        out[k] = lo; out[k | dist] = hi;
      }
    }
  }
}

// the two runs that meet at merged position `at` of a list whose runs of `run_len` entries are
// merged pairwise: returns the position inside the pair
__device__ __forceinline__ int merge_pair(const float *list, long long rows, long long run_len, long long at,
                                          const float *&left, int &la, const float *&right, int &lb) {
  const long long start = at / (2 * run_len) * (2 * run_len);
  const long long left_len = rows - start < run_len ? rows - start : run_len;
  const long long right_len = rows - start - left_len < run_len ? rows - start - left_len : run_len;
  left = list + start; la = (int)left_len;
  right = left + left_len; lb = (int)right_len;
  return (int)(at - start);
}

// one round that is not the last: runs of run_len entries become runs of twice that
__global__ void __launch_bounds__(kSwdW1Threads)
swd_merge_kernel(const float *in, float *out, long long rows, long long run_len, int lists, const int *skip,
                 const SwdExtents ext) {
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const long long spans = (rows + kSwdMergeSpan - 1) / kSwdMergeSpan;
  const long long task = (long long)blockIdx.x * kSwdW1Threads + threadIdx.x;
  if (task >= spans * lists) return;
  const long long list = task / spans, at = (task - list * spans) * kSwdMergeSpan;
  const float *left, *right;
  int la, lb;
  // (a span may straddle two pairs only if 2 * run_len is not a multiple of the span: run_len is a multiple of T, any T,
  // so the entries past the end of this pair are produced one by one below)
  const int d = merge_pair(in + list * rows, rows, run_len, at, left, la, right, lb);
  // the pair's two runs and this thread's outputs lie inside the list, the list inside the buffer
  if (!SENTINEL_BOUNDS(kSiteSwdLists, left - in, la + lb, ext.list_floats) ||
      !SENTINEL_BOUNDS(kSiteSwdLists, list * rows + at, (rows - at < kSwdMergeSpan ? rows - at : kSwdMergeSpan), ext.list_floats))
    return;
  float v[kSwdMergeSpan];
  merge_span(left, la, right, lb, d, v);
  float *dst = out + list * rows + at;
  const int n_here = la + lb - d < kSwdMergeSpan ? la + lb - d : kSwdMergeSpan;
#pragma unroll
  for (int k = 0; k < kSwdMergeSpan; ++k)
    if (k < n_here) dst[k] = v[k];
  if (n_here < kSwdMergeSpan) {                   // the rest of the span lies in the next pair (or past the end)
    for (int k = n_here; k < kSwdMergeSpan && at + k < rows; ++k) {
      const float *l2, *r2;
      int la2, lb2;
      const int d2 = merge_pair(in + list * rows, rows, run_len, at + k, l2, la2, r2, lb2);
      float w[kSwdMergeSpan];
      merge_span(l2, la2, r2, lb2, d2, w);
      dst[k] = w[0];
    }
  }
}

__host__ __device__ inline int swd_w1_chunks(long long n) { return (int)((n + kSwdW1Span - 1) / kSwdW1Span); }
// doubles of `partial`: per direction the whole-tensor CTAs' sums, then per (direction, sample) the sample CTAs'
__host__ __device__ inline size_t swd_w1_partials(int L, int B, int T) {
  return (size_t)L * swd_w1_chunks((long long)B * T) + (size_t)L * B * swd_w1_chunks(T);
}

// `sorted`: the samples' sorted lists, [2L][B][T]; `runs`: the lists after all merge rounds but the last
// (runs of run_len entries; == sorted if there was no earlier round; unused if B == 1)
__global__ void __launch_bounds__(kSwdW1Threads)
swd_w1_kernel(const float *sorted, const float *runs, long long run_len, double *partial, unsigned *ticket, float *out, int B,
              int T, int L, long long rows, const int *skip, const SwdExtents ext) {
  __shared__ double s_red[kSwdW1Threads / 32];
  __shared__ float s_w1[(kMaxB + 1) * 16];        // W1 per (unit, direction), L <= 16
  __shared__ bool s_last;
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const int tensor_chunks = B > 1 ? swd_w1_chunks(rows) : 0, sample_chunks = swd_w1_chunks(T);
  const int n_tensor = L * tensor_chunks;
  double term = 0.;
  if ((int)blockIdx.x < n_tensor) {               // a span of the last merge round, both clouds
    const int l = blockIdx.x / tensor_chunks, chunk = blockIdx.x - l * tensor_chunks;
    const long long at = ((long long)chunk * kSwdW1Threads + threadIdx.x) * kSwdMergeSpan;
    if (at < rows && SENTINEL_BOUNDS(kSiteSwdLists, ((size_t)L + l) * rows, rows, ext.list_floats)) {   // (both clouds' lists of direction l)
      float va[kSwdMergeSpan], vb[kSwdMergeSpan];
      const float *left, *right;
      int la, lb;
      int d = merge_pair(runs + (size_t)l * rows, rows, run_len, at, left, la, right, lb);
      merge_span(left, la, right, lb, d, va);
      d = merge_pair(runs + ((size_t)L + l) * rows, rows, run_len, at, left, la, right, lb);
      merge_span(left, la, right, lb, d, vb);
#pragma unroll
      for (int k = 0; k < kSwdMergeSpan; ++k)
        if (at + k < rows) term += (double)fabsf(va[k] - vb[k]);
    }
  } else {                                        // a span of one sample's two lists
    const int unit = (blockIdx.x - n_tensor) / sample_chunks, chunk = (blockIdx.x - n_tensor) - unit * sample_chunks;
    const int l = unit / B, b = unit - l * B;
    const float *sa = sorted + (size_t)l * rows + (size_t)b * T, *sb = sorted + ((size_t)L + l) * rows + (size_t)b * T;
    const int at = (chunk * kSwdW1Threads + threadIdx.x) * kSwdMergeSpan;
    const bool inside = SENTINEL_BOUNDS(kSiteSwdLists, ((size_t)L + l) * rows + (size_t)b * T, T, ext.list_floats);
#pragma unroll
    for (int k = 0; k < kSwdMergeSpan; ++k)
      if (inside && at + k < T) term += (double)fabsf(sa[at + k] - sb[at + k]);
  }
  const double sum = block_sum_ordered(term, s_red);
  if (threadIdx.x == 0) {
    if (SENTINEL_BOUNDS(kSiteSwdPartial, blockIdx.x, 1, ext.partial_doubles)) partial[blockIdx.x] = sum;
    __threadfence();
    s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // unit r = 0: the whole tensor, r = 1 + b: sample b.  One warp per (unit, direction): lane j adds
  // the CTA sums j, j + 32, ... in that order, the lanes are combined by the shuffle tree
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int pair = warp; pair < (B + 1) * L; pair += kSwdW1Threads / 32) {
    const int r = pair / L, dir = pair - r * L;
    double w1 = 0., n = (double)T;
    if (r == 0 && B > 1) {
      for (int k = lane; k < tensor_chunks; k += 32) w1 += __ldcg(partial + (size_t)dir * tensor_chunks + k);
      n = (double)rows;
    } else {
      const int bb = r == 0 ? 0 : r - 1;
      for (int k = lane; k < sample_chunks; k += 32) w1 += __ldcg(partial + n_tensor + ((size_t)dir * B + bb) * sample_chunks + k);
    }
    w1 = warp_sum(w1);
    if (lane == 0) s_w1[pair] = (float)(w1 / n);
  }
  __syncthreads();
  // a sample with an entry that is not finite has a W1 that is not finite (inf, or inf - inf); the
  // whole tensor's W1 is declared not a number along with it, whatever the merged lists gave
  for (int r = threadIdx.x; r <= B; r += kSwdW1Threads) {
    double mean = 0.;
    for (int dir = 0; dir < L; ++dir) mean += (double)s_w1[r * L + dir];
    if (r == 0) {
      bool finite = true;
      for (int k = L; k < (B + 1) * L; ++k) finite = finite && fabsf(s_w1[k]) < CUDART_INF_F;
      if (!finite) mean = (double)CUDART_NAN_F;
    }
    out[r] = (float)(mean / L);
  }
}

}  // namespace sentinel
