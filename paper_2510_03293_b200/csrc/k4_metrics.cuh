// K4: imbalance figures from the dispatch offsets of a finished call (Motivation: imbalance
// of experts and of devices under a placement).
//   N_e     = offsets[e+1] - offsets[e]          assignments of expert e in this layer
//   I_L     = max_e N_e / mean_e N_e
//   N_g     = sum_e A[g,e] N_e                   A >= 0 with unit column sums (replication
//                                                splits an expert's tokens), or 0/1 through an
//                                                expert -> bin map, or contiguous blocks
//   I_bins  = max_g N_g / mean_g N_g
//   I_agg   = sum_L w_L I_L,  w_L = assignments of layer L / all assignments
// k4_imbalance: one block per layer (grid-stride).  Counts are exact integers, bin loads and
// ratios are formed in fp64 and rounded once to fp32.  k4_aggregate: one block, fixed
// reduction order, so results do not depend on scheduling.
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK4Threads = 256;
constexpr int kK4MaxBins = 1024;

__device__ __forceinline__ double k4_warp_sum(double v) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
  return v;
}
__device__ __forceinline__ double k4_warp_max(double v) {
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, s));
  return v;
}

// Block-wide (sum, max) of one value per thread; every thread gets the result.
__device__ __forceinline__ void k4_block_sum_max(double& sum, double& mx, double* red) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  sum = k4_warp_sum(sum);
  mx = k4_warp_max(mx);
  __syncthreads();
  if (lane == 0) { red[warp] = sum; red[8 + warp] = mx; }
  __syncthreads();
  sum = 0.0;
  mx = 0.0;
  for (int w = 0; w < kK4Threads / 32; ++w) { sum += red[w]; mx = fmax(mx, red[8 + w]); }
}

__global__ void __launch_bounds__(kK4Threads)
k4_imbalance(int n_layers, int E, int n_bins, const int32_t* __restrict__ offsets,
             const int32_t* __restrict__ e2b, const float* __restrict__ placement,
             float* imbalance, float* bin_imbalance) {
  __shared__ int32_t s_cnt[kMaxExperts];
  __shared__ int32_t s_ibin[kMaxExperts];
  __shared__ double s_bin[kK4MaxBins];
  __shared__ double s_red[16];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int per = (E + n_bins - 1) / n_bins;
  for (int l = blockIdx.x; l < n_layers; l += gridDim.x) {
    const int32_t* off = offsets + (size_t)l * (E + 1);
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += kK4Threads) s_cnt[e] = off[e + 1] - off[e];
    if (!placement)
      for (int b = threadIdx.x; b < n_bins; b += kK4Threads) s_ibin[b] = 0;
    __syncthreads();
    double sum = 0.0, mx = 0.0;
    for (int e = threadIdx.x; e < E; e += kK4Threads) {
      sum += (double)s_cnt[e];
      mx = fmax(mx, (double)s_cnt[e]);
    }
    k4_block_sum_max(sum, mx, s_red);
    if (threadIdx.x == 0) imbalance[l] = sum > 0.0 ? (float)(mx * (double)E / sum) : 1.0f;
    if (!bin_imbalance) continue;

    if (placement) {
      for (int g = warp; g < n_bins; g += kK4Threads / 32) {
        double acc = 0.0;
        for (int e = lane; e < E; e += 32) acc += (double)placement[(size_t)g * E + e] * s_cnt[e];
        acc = k4_warp_sum(acc);
        if (lane == 0) s_bin[g] = acc;
      }
    } else {
      for (int e = threadIdx.x; e < E; e += kK4Threads) {
        // an expert mapped outside [0, n_bins) belongs to no bin, as in the routing kernel
        const int b = e2b ? e2b[e] : e / per;
        if (b >= 0 && b < n_bins) atomicAdd(&s_ibin[b], s_cnt[e]);
      }
      __syncthreads();
      for (int b = threadIdx.x; b < n_bins; b += kK4Threads) s_bin[b] = (double)s_ibin[b];
    }
    __syncthreads();
    double bsum = 0.0, bmx = 0.0;
    for (int b = threadIdx.x; b < n_bins; b += kK4Threads) {
      bsum += s_bin[b];
      bmx = fmax(bmx, s_bin[b]);
    }
    k4_block_sum_max(bsum, bmx, s_red);
    if (threadIdx.x == 0)
      bin_imbalance[l] = bsum > 0.0 ? (float)(bmx * (double)n_bins / bsum) : 1.0f;
  }
}

// aggregate[0] = sum_L w_L I_L, aggregate[1] = the same over bin_imbalance (1 if absent).
__global__ void __launch_bounds__(kK4Threads)
k4_aggregate(int n_layers, int E, const int32_t* __restrict__ offsets,
             const float* __restrict__ imbalance, const float* __restrict__ bin_imbalance,
             float* aggregate) {
  __shared__ double s_part[3][kK4Threads];
  double a = 0.0, b = 0.0, d = 0.0;
  for (int l = threadIdx.x; l < n_layers; l += kK4Threads) {
    const int32_t* off = offsets + (size_t)l * (E + 1);
    const double tot = (double)(off[E] - off[0]);
    a += tot * (double)imbalance[l];
    b += tot * (double)(bin_imbalance ? bin_imbalance[l] : 1.0f);
    d += tot;
  }
  s_part[0][threadIdx.x] = a;
  s_part[1][threadIdx.x] = b;
  s_part[2][threadIdx.x] = d;
  __syncthreads();
  for (int s = kK4Threads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s)
      for (int q = 0; q < 3; ++q) s_part[q][threadIdx.x] += s_part[q][threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double den = s_part[2][0];
    // no assignment at all: every layer reports 1, and so does the aggregate
    aggregate[0] = den > 0.0 ? (float)(s_part[0][0] / den) : 1.0f;
    aggregate[1] = den > 0.0 ? (float)(s_part[1][0] / den) : 1.0f;
  }
}

}  // namespace laser
