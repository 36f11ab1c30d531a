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

// one CTA per (sample, direction, cloud): bitonic sort of that list of T projections in shared
// memory (padded with +inf to a power of two, at least 8); the sorted list goes back to global
// memory
__global__ void __launch_bounds__(kSwdSortThreads)
swd_sort_samples_kernel(const float *proj, float *sorted, int B, int T, int L, long long rows, const int *skip) {
  extern __shared__ float s_val[];                // [npad]
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const int list = blockIdx.x / B, b = blockIdx.x - list * B;     // list = cloud * L + direction
  int npad = 8;
  while (npad < T) npad <<= 1;
  const float *src = proj + (size_t)list * rows + (size_t)b * T;
  for (int i = threadIdx.x; i < npad; i += kSwdSortThreads) s_val[i] = i < T ? src[i] : CUDART_INF_F;
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
  float *dst = sorted + (size_t)list * rows + (size_t)b * T;
  for (int i = threadIdx.x; i < T; i += kSwdSortThreads) dst[i] = s_val[i];
}

// per sample and direction: W1 = mean |a_(i) - b_(i)| of the two sorted lists
__global__ void __launch_bounds__(256)
swd_sample_w1_kernel(const float *sorted, float *w1_sample, int B, int T, int L, long long rows, const int *skip) {
  __shared__ double s_red[256 / 32];
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const int b = blockIdx.x / L, l = blockIdx.x - b * L;
  const float *sa = sorted + (size_t)l * rows + (size_t)b * T;
  const float *sb = sorted + ((size_t)L + l) * rows + (size_t)b * T;
  double acc = 0.;
  for (int i = threadIdx.x; i < T; i += 256) acc += (double)fabsf(sa[i] - sb[i]);
  const double total = block_sum_ordered(acc, s_red);
  if (threadIdx.x == 0) w1_sample[b * L + l] = (float)(total / (double)T);
}

// ---------------------------------------------------------------------------------------------
// one round of merging: in every list (2L of them, each B sorted runs of T) neighbouring pairs
// of runs of `run` samples become one sorted run; an element's place is its index in its own
// run plus its rank in the partner run (left run first on ties)
__global__ void swd_merge_kernel(const float *in, float *out, long long rows, int T, int run, int lists,
                                 const int *skip) {
  chain_entry();
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * lists || (skip && __ldcg(skip))) return;
  const long long list = e / rows, i = e - list * rows;
  const float *src = in + list * rows;
  const long long run_len = (long long)run * T;
  const long long r = i / run_len, pair_start = (r & ~1ll) * run_len;
  const long long own_start = r * run_len;
  const long long other_start = (r & 1) ? own_start - run_len : own_start + run_len;
  const float v = src[i];
  long long pos = i - own_start;
  if (other_start < rows) {
    long long lo = 0, hi = run_len;
    if (other_start + hi > rows) hi = rows - other_start;
    const float *other = src + other_start;
    if (r & 1) {                                  // right run: after the left entries <= v
      while (lo < hi) { const long long mid = (lo + hi) >> 1; if (other[mid] <= v) lo = mid + 1; else hi = mid; }
    } else {                                      // left run: after the right entries < v
      while (lo < hi) { const long long mid = (lo + hi) >> 1; if (other[mid] < v) lo = mid + 1; else hi = mid; }
    }
    pos += lo;
  }
  out[list * rows + pair_start + pos] = v;
}

// whole-tensor unit: W1 per direction from the fully merged lists, one CTA per direction
__global__ void __launch_bounds__(kSwdSortThreads)
swd_tensor_w1_kernel(const float *merged, float *w1_tensor, long long rows, int L, const int *skip) {
  __shared__ double s_red[kSwdSortThreads / 32];
  chain_entry();
  if (skip && __ldcg(skip)) return;
  const int l = blockIdx.x;
  const float *a = merged + (size_t)l * rows, *b = merged + ((size_t)L + l) * rows;
  double acc = 0.;
  for (long long i = threadIdx.x; i < rows; i += kSwdSortThreads) acc += (double)fabsf(a[i] - b[i]);
  const double total = block_sum_ordered(acc, s_red);
  if (threadIdx.x == 0) w1_tensor[l] = (float)(total / (double)rows);
}

// the means over the directions for every unit: out[0] = tensor, out[1+b] = sample b
__global__ void swd_finish_kernel(const float *w1_tensor, const float *w1_sample, float *out, int B, int L,
                                  const int *skip) {
  chain_entry();
  if (skip && __ldcg(skip)) return;
  for (int r = threadIdx.x; r <= B; r += blockDim.x) {
    const float *w = r ? w1_sample + (size_t)(r - 1) * L : w1_tensor;
    double s = 0.;
    for (int l = 0; l < L; ++l) s += (double)w[l];
    out[r] = (float)(s / L);
  }
}

}  // namespace sentinel
