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
constexpr int kSwdMaxTokensPerSample = 16384;    // one sample's projections are sorted in shared memory

// ---------------------------------------------------------------------------------------------
// projections: proj[(t*L + l)*rows + row] = sum_c v[row][c] * u[l][c], t = 0 for x, 1 for m.
// A warp owns whole rows; the directions sit in shared memory as bf16 (they are given as bf16).
// Traffic: x and m are read once, 6 B/element; per element L multiply-adds for each of x and m.
// The reference is m1 if *active is non-zero, else m0 (a verifier keeps two buffers and flips
// between them on the device); every kernel of the chain returns at once if *skip is non-zero
// (a banned worker's tensor is not read).  Both pointers may be nullptr.
//
// Projection is linear and so is Eq. 1: the projections of the reference obey
//   P(m_t) = beta P(m_{t-1}) + (1-beta) P(x_t)
// whenever the reference moves.  A verifier therefore keeps P(m) itself ([rows][L] doubles, two
// buffers pm0 / pm1 selected by the same `active` word as the reference, so a step that does not
// commit leaves them alone): this kernel always writes the candidate P(m_t) into the spare one,
// and with kIncr = true it takes P(m_{t-1}) from the current one instead of reading m at all --
// 2 B/element of traffic instead of 6.  kIncr = false computes it from m (and stores it, if
// the buffers are given): the stateless call, and the first step after a state import.
template <int L, int kSwdThreads, bool kIncr>
__global__ void __launch_bounds__(kSwdThreads, kSwdThreads == 512 ? 2 : 1)
swd_project_kernel(const uint16_t *x, const float *m0, const float *m1, const int *active, const int *skip,
                   const uint16_t *u, float *proj, long long rows, int d, double *pm0, double *pm1, float beta,
                   float one_minus_beta) {
  extern __shared__ uint4 s_u[];                 // [L][d/8], 8 bf16 each
  if (skip && __ldcg(skip)) return;
  const bool second = active && __ldcg(active);
  const float *m = second ? m1 : m0;
  double *pm_cur = second ? pm1 : pm0, *pm_next = second ? pm0 : pm1;
  const int chunks = d >> 3;
  for (int i = threadIdx.x; i < L * chunks; i += kSwdThreads)
    s_u[i] = reinterpret_cast<const uint4 *>(u)[i];
  __syncthreads();

  // A warp owns kRows whole rows at a time; with two rows every direction word fetched from shared
  // memory serves both (without the reference to read, shared memory is the busier path).
  constexpr int kRows = (kIncr && L <= 8) ? 2 : 1;     // (16 directions leave no registers for a second row)
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (kSwdThreads / 32) + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * (kSwdThreads / 32);
  for (long long row0 = warp * kRows; row0 < rows; row0 += n_warps * kRows) {
    float ax[kRows][L], am[L];
#pragma unroll
    for (int l = 0; l < L; ++l) {
      am[l] = 0.f;
#pragma unroll
      for (int r = 0; r < kRows; ++r) ax[r][l] = 0.f;
    }
    bool live[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) live[r] = row0 + r < rows;
    const size_t off = (size_t)row0 * d;
    // two chunks per trip, their loads issued before any arithmetic (more bytes in flight)
    for (int c0 = lane; c0 < chunks; c0 += 64) {
      uint4 xv[kRows][2];
      F8 mv[2];
      bool ok[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = c0 + 32 * h;
        ok[h] = c < chunks;
        if (ok[h]) {
#pragma unroll
          for (int r = 0; r < kRows; ++r)
            if (live[r]) xv[r][h] = ld_x128(x + off + (size_t)r * d + (size_t)c * 8);
          if (!kIncr) mv[h] = ld_m256(m + off + (size_t)c * 8);
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (!ok[h]) continue;
        const int c = c0 + 32 * h;
        float xf[kRows][8];
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          const unsigned xw[4] = {xv[r][h].x, xv[r][h].y, xv[r][h].z, xv[r][h].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            xf[r][2 * j] = live[r] ? __uint_as_float(xw[j] << 16) : 0.f;
            xf[r][2 * j + 1] = live[r] ? __uint_as_float(xw[j] & 0xFFFF0000u) : 0.f;
          }
        }
#pragma unroll
        for (int l = 0; l < L; ++l) {
          const uint4 uv = s_u[l * chunks + c];
          const unsigned uw[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float u_lo = __uint_as_float(uw[j] << 16), u_hi = __uint_as_float(uw[j] & 0xFFFF0000u);
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
              ax[r][l] = fmaf(xf[r][2 * j], u_lo, ax[r][l]);
              ax[r][l] = fmaf(xf[r][2 * j + 1], u_hi, ax[r][l]);
            }
            if (!kIncr) {
              am[l] = fmaf(mv[h].v[2 * j], u_lo, am[l]);
              am[l] = fmaf(mv[h].v[2 * j + 1], u_hi, am[l]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const long long row = row0 + r;
#pragma unroll
      for (int l = 0; l < L; ++l) {
        const float sx = warp_sum(ax[r][l]);
        const float sm = kIncr ? 0.f : warp_sum(am[l]);
        if (lane == l && live[r]) {
          const size_t at = (size_t)row * L + l;
          const double p_cur = kIncr ? pm_cur[at] : (double)sm;
          proj[(size_t)l * rows + row] = sx;
          proj[((size_t)L + l) * rows + row] = (float)p_cur;
          if (pm_cur) {
            if (!kIncr) pm_cur[at] = p_cur;
            pm_next[at] = (double)beta * p_cur + (double)one_minus_beta * (double)sx;
          }
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

// one CTA per (sample, direction, cloud): bitonic sort of that list of T projections in shared
// memory; the sorted list goes back to global memory
__global__ void __launch_bounds__(kSwdSortThreads)
swd_sort_samples_kernel(const float *proj, float *sorted, int B, int T, int L, long long rows, const int *skip) {
  extern __shared__ float s_val[];                // [npad]
  if (skip && __ldcg(skip)) return;
  const int list = blockIdx.x / B, b = blockIdx.x - list * B;     // list = cloud * L + direction
  int npad = 1;
  while (npad < T) npad <<= 1;
  const float *src = proj + (size_t)list * rows + (size_t)b * T;
  for (int i = threadIdx.x; i < npad; i += kSwdSortThreads) s_val[i] = i < T ? src[i] : CUDART_INF_F;
  __syncthreads();
  for (int k2 = 2; k2 <= npad; k2 <<= 1) {        // bitonic sort, ascending
    for (int j2 = k2 >> 1; j2 > 0; j2 >>= 1) {
      for (int t = threadIdx.x; t < npad; t += kSwdSortThreads) {
        const int partner = t ^ j2;
        if (partner > t) {
          const bool up = ((t & k2) == 0);
          const float a0 = s_val[t], a1 = s_val[partner];
          if ((a0 > a1) == up) { s_val[t] = a1; s_val[partner] = a0; }
        }
      }
      __syncthreads();
    }
  }
  float *dst = sorted + (size_t)list * rows + (size_t)b * T;
  for (int i = threadIdx.x; i < T; i += kSwdSortThreads) dst[i] = s_val[i];
}

// per sample and direction: W1 = mean |a_(i) - b_(i)| of the two sorted lists
__global__ void __launch_bounds__(256)
swd_sample_w1_kernel(const float *sorted, float *w1_sample, int B, int T, int L, long long rows, const int *skip) {
  __shared__ double s_red[256 / 32];
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
  if (skip && __ldcg(skip)) return;
  for (int r = threadIdx.x; r <= B; r += blockDim.x) {
    const float *w = r ? w1_sample + (size_t)(r - 1) * L : w1_tensor;
    double s = 0.;
    for (int l = 0; l < L; ++l) s += (double)w[l];
    out[r] = (float)(s / L);
  }
}

}  // namespace sentinel
