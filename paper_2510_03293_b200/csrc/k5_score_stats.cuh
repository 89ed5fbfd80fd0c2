// K5: gate-score statistics of a batch, per layer, from fp32 logits (Layer Variability in Gate
// Score Distributions: top-k mass, entropy, routing regimes) -- the figures from which the
// dominance cutoff and the pool threshold are chosen per layer.
//
// Eight lanes share a token (lane j holds experts j, j+8, ...), which is also the summation
// layout of the routing softmax: Z, the scores and M_k come out bit for bit as in the router.
// Per token:
//   M_k     k rounds of "best remaining" by (logit descending, index ascending), scores added
//           left to right in fp32
//   H       -sum_i s_i ln s_i in fp64 (nats)
//   n_near  #{i : s_i >= fl32(near_ratio * s_max)}; regime 0 (single-head) if 1, 1 (plateau)
//           if <= plateau_max, else 2 (smooth)
// Accumulation is in 64-bit integers (per thread in registers over its tokens, then per block in
// shared memory, then one global atomic per word and block; the histogram in 32-bit shared
// counters), so the sums do not depend on the order of arrival: M_k and s_max are fp32
// values >= 2^-9, hence exact multiples of 2^-32; H is rounded to the nearest 2^-32.
//   word 0 tokens | 1 sum M_k 2^32 | 2 sum H 2^32 | 3..5 regime counts | 6 sum n_near |
//   7 sum s_max 2^32 | 8..71 histogram of M_k over 64 equal bins of [0,1]
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kStatsWords = 72;
constexpr int kStatsThreads = 256;

template <int N>
__global__ void __launch_bounds__(kStatsThreads)
k5_score_stats(int T, int E, int k, const float* __restrict__ logits, float near_ratio,
               int plateau_max, unsigned long long* __restrict__ stats) {
  constexpr int EPL = N / 8;
  __shared__ unsigned long long s_acc[8];
  __shared__ unsigned int s_hist[64];
  const int layer = blockIdx.y;
  const float* X = logits + (size_t)layer * T * E;
  if (threadIdx.x < 8) s_acc[threadIdx.x] = 0ull;
  if (threadIdx.x < 64) s_hist[threadIdx.x] = 0u;
  __syncthreads();
  unsigned long long acc[8] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
  const int j = threadIdx.x & 7;
  const float ninf = __int_as_float(0xff800000);
  constexpr int TPB = kStatsThreads / 8;   // tokens per block and pass

  for (long long t0 = (long long)blockIdx.x * TPB; t0 < T; t0 += (long long)gridDim.x * TPB) {
    const long long tt = t0 + (threadIdx.x >> 3);
    const bool valid = tt < T;
    const float* row = X + (size_t)(valid ? tt : T - 1) * E;   // idle groups redo the last token
    float x[EPL];
    float xmax = ninf;
#pragma unroll
    for (int m = 0; m < EPL; ++m) {
      const int i = 8 * m + j;
      x[m] = i < E ? row[i] : ninf;
      xmax = fmaxf(xmax, x[m]);
    }
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) xmax = fmaxf(xmax, __shfl_xor_sync(0xffffffffu, xmax, s));
    float e[EPL];
    float a = 0.0f;
#pragma unroll
    for (int m = 0; m < EPL; ++m) {
      e[m] = 8 * m + j < E ? exp32(__fsub_rn(x[m], xmax)) : 0.0f;
      if (8 * m + j < E) a = __fadd_rn(a, e[m]);
    }
    float Z = a;
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) Z = __fadd_rn(Z, __shfl_xor_sync(0xffffffffu, Z, s));

    // M_k: k rounds of "best remaining"
    float prev_x = __int_as_float(0x7f800000);
    int prev_i = -1;
    float Mk = 0.0f, smax = 0.0f;
#pragma unroll 1
    for (int r = 0; r < k; ++r) {
      float bx = ninf;
      int bi = 0x7fffffff;
#pragma unroll
      for (int m = 0; m < EPL; ++m) {
        const int i = 8 * m + j;
        const float xi = x[m];
        const bool after_prev = (xi < prev_x) || (xi == prev_x && i > prev_i);
        if (i < E && after_prev && xi > bx) { bx = xi; bi = i; }
      }
#pragma unroll
      for (int s = 1; s < 8; s <<= 1) {
        const float ox = __shfl_xor_sync(0xffffffffu, bx, s);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
        if (ox > bx || (ox == bx && oi < bi)) { bx = ox; bi = oi; }
      }
      const float sr = __fdiv_rn(exp32(__fsub_rn(bx, xmax)), Z);
      if (r == 0) { Mk = sr; smax = sr; }
      else Mk = __fadd_rn(Mk, sr);
      prev_x = bx;
      prev_i = bi;
    }
    // entropy and the number of experts near the top
    const float thr = __fmul_rn(near_ratio, smax);
    double h = 0.0;
    int near = 0;
#pragma unroll
    for (int m = 0; m < EPL; ++m) {
      if (8 * m + j < E) {
        const float s = __fdiv_rn(e[m], Z);
        if (s > 0.0f) h -= (double)s * log((double)s);
        near += s >= thr ? 1 : 0;
      }
    }
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) {
      h += __shfl_xor_sync(0xffffffffu, h, s);
      near += __shfl_xor_sync(0xffffffffu, near, s);
    }
    if (valid && j == 0) {
      const int regime = near == 1 ? 0 : (near <= plateau_max ? 1 : 2);
      int bin = (int)(Mk * 64.0f);   // exact product; M_k can round to just above 1
      bin = bin > 63 ? 63 : bin;
      acc[0] += 1ull;
      acc[1] += (unsigned long long)((double)Mk * 4294967296.0);
      acc[2] += (unsigned long long)(fmax(h, 0.0) * 4294967296.0 + 0.5);
      acc[3] += regime == 0 ? 1ull : 0ull;
      acc[4] += regime == 1 ? 1ull : 0ull;
      acc[5] += regime == 2 ? 1ull : 0ull;
      acc[6] += (unsigned long long)near;
      acc[7] += (unsigned long long)((double)smax * 4294967296.0);
      atomicAdd(&s_hist[bin], 1u);
    }
  }
  // the warp's four token lanes (0, 8, 16, 24) -> lane 0 -> block
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], 8);
    acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], 16);
    if ((threadIdx.x & 31) == 0 && acc[q]) atomicAdd(&s_acc[q], acc[q]);
  }
  __syncthreads();
  unsigned long long* out = stats + (size_t)layer * kStatsWords;
  if (threadIdx.x < 8 && s_acc[threadIdx.x]) atomicAdd(&out[threadIdx.x], s_acc[threadIdx.x]);
  if (threadIdx.x >= 64 && threadIdx.x < 128 && s_hist[threadIdx.x - 64])
    atomicAdd(&out[8 + threadIdx.x - 64], (unsigned long long)s_hist[threadIdx.x - 64]);
}

// means[l] = (mean M_k, mean entropy in nats, mean s_max, mean n_near); zeros without tokens.
__global__ void k5_stats_means(int n_layers, const unsigned long long* __restrict__ stats,
                               float* __restrict__ means) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= n_layers) return;
  const unsigned long long* w = stats + (size_t)l * kStatsWords;
  const double n = (double)w[0];
  const double q = 1.0 / 4294967296.0;
  means[4 * l + 0] = n > 0 ? (float)((double)w[1] * q / n) : 0.0f;
  means[4 * l + 1] = n > 0 ? (float)((double)w[2] * q / n) : 0.0f;
  means[4 * l + 2] = n > 0 ? (float)((double)w[7] * q / n) : 0.0f;
  means[4 * l + 3] = n > 0 ? (float)((double)w[6] / n) : 0.0f;
}

}  // namespace laser
