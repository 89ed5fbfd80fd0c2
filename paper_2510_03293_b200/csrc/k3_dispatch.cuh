// K3: expert dispatch from the chosen expert ids -- per-call counts, exclusive offsets, the
// stable grouping of pair ids t*k+j by expert -- and device-bin load sums (N_g = sum of the
// counts of the experts placed on bin g).  Three passes, none of which uses an atomic:
//   k3_hist    block histograms from warp-private counters (match-any + leader add)
//   k3_scan    per-expert prefix over blocks, warp-scan prefix over experts, bin sums
//   k3_scatter stable scatter with warp-private running bases
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK3Threads = 256;
constexpr int kK3Warps = kK3Threads / 32;
constexpr int kK3PairsPerWarp = kDispatchPairsPerBlock / kK3Warps;

// Counts the experts of this warp's contiguous span of pair ids into hist (warp-private).
__device__ __forceinline__ void k3_warp_hist(const int32_t* __restrict__ ids, long long begin,
                                             long long end, int32_t* hist, int lane) {
  for (long long p0 = begin; p0 < end; p0 += 32) {
    const long long p = p0 + lane;
    const int e = p < end ? ids[p] : -1;
    const unsigned same = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && (same & ((1u << lane) - 1)) == 0) hist[e] += __popc(same);
    __syncwarp();
  }
}

__global__ void __launch_bounds__(kK3Threads) k3_hist(const RouteArgs A) {
  extern __shared__ int32_t k3_smem[];  // [kK3Warps][E]
  const int layer = A.layer0 + blockIdx.y;
  const int E = A.E, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long n = (long long)A.T * A.k;
  const int32_t* ids = A.expert_ids + (size_t)layer * n;
  for (int i = tid; i < kK3Warps * E; i += kK3Threads) k3_smem[i] = 0;
  __syncthreads();
  const long long begin = min(n, (long long)blockIdx.x * kDispatchPairsPerBlock +
                                     (long long)warp * kK3PairsPerWarp);
  const long long end = min(n, begin + kK3PairsPerWarp);
  k3_warp_hist(ids, begin, end, k3_smem + warp * E, lane);
  __syncthreads();
  int32_t* blk = reinterpret_cast<int32_t*>(A.ws + (size_t)layer * A.ws_ls + A.lay.blk_hist) +
                 (size_t)blockIdx.x * E;
  for (int e = tid; e < E; e += kK3Threads) {
    int32_t s = 0;
#pragma unroll
    for (int w = 0; w < kK3Warps; ++w) s += k3_smem[w * E + e];
    blk[e] = s;
  }
}

// One block per layer.  Turns block histograms into block bases (global positions), writes
// offsets[E+1] and adds the per-bin sums of this call's counts to bin_loads.
__global__ void __launch_bounds__(kK3Threads) k3_scan(const RouteArgs A) {
  __shared__ int32_t counts[kMaxExperts];
  __shared__ int32_t excl[kMaxExperts];
  __shared__ int32_t warp_tot[kK3Warps];
  const int layer = A.layer0 + blockIdx.x;
  const int E = A.E, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int32_t* blk = reinterpret_cast<int32_t*>(A.ws + (size_t)layer * A.ws_ls + A.lay.blk_hist);
  const int n_blk = A.lay.n_blk;

  int32_t total = 0;
  if (tid < E) {
    for (int b = 0; b < n_blk; ++b) {
      const int32_t v = blk[(size_t)b * E + tid];
      blk[(size_t)b * E + tid] = total;
      total += v;
    }
    counts[tid] = total;
  }
  // exclusive prefix over experts: inclusive warp scan by shuffles, then warp totals
  int32_t incl = total;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const int32_t up = __shfl_up_sync(0xffffffffu, incl, s);
    if (lane >= s) incl += up;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int32_t base = 0;
  for (int w = 0; w < warp; ++w) base += warp_tot[w];
  if (tid < E) excl[tid] = base + incl - total;
  __syncthreads();

  int32_t* offsets = A.offsets + (size_t)layer * (E + 1);
  if (tid < E) {
    offsets[tid] = excl[tid];
    if (tid == E - 1) offsets[E] = excl[tid] + total;
    for (int b = 0; b < n_blk; ++b) blk[(size_t)b * E + tid] += excl[tid];
  }
  if (A.bin_loads) {
    const int B = A.n_bins;
    const int per = (E + B - 1) / B;
    int32_t* bl = A.bin_loads + (size_t)layer * B;
    for (int b = tid; b < B; b += kK3Threads) {
      int32_t s = 0;
      for (int e = 0; e < E; ++e) {
        const int be = A.e2b ? A.e2b[e] : e / per;
        if (be == b) s += counts[e];
      }
      bl[b] += s;
    }
  }
}

__global__ void __launch_bounds__(kK3Threads) k3_scatter(const RouteArgs A) {
  extern __shared__ int32_t k3_smem[];  // [kK3Warps][E] histograms, then running bases
  const int layer = A.layer0 + blockIdx.y;
  const int E = A.E, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long n = (long long)A.T * A.k;
  const int32_t* ids = A.expert_ids + (size_t)layer * n;
  int32_t* perm = A.perm + (size_t)layer * n;
  for (int i = tid; i < kK3Warps * E; i += kK3Threads) k3_smem[i] = 0;
  __syncthreads();
  const long long begin = min(n, (long long)blockIdx.x * kDispatchPairsPerBlock +
                                     (long long)warp * kK3PairsPerWarp);
  const long long end = min(n, begin + kK3PairsPerWarp);
  k3_warp_hist(ids, begin, end, k3_smem + warp * E, lane);
  __syncthreads();
  const int32_t* blk = reinterpret_cast<const int32_t*>(A.ws + (size_t)layer * A.ws_ls +
                                                         A.lay.blk_hist) + (size_t)blockIdx.x * E;
  for (int e = tid; e < E; e += kK3Threads) {
    int32_t run = blk[e];
#pragma unroll
    for (int w = 0; w < kK3Warps; ++w) {
      const int32_t h = k3_smem[w * E + e];
      k3_smem[w * E + e] = run;
      run += h;
    }
  }
  __syncthreads();
  int32_t* base = k3_smem + warp * E;
  for (long long p0 = begin; p0 < end; p0 += 32) {
    const long long p = p0 + lane;
    const int e = p < end ? ids[p] : -1;
    const unsigned same = __match_any_sync(0xffffffffu, e);
    const unsigned before = same & ((1u << lane) - 1);
    if (e >= 0) perm[base[e] + __popc(before)] = (int32_t)p;
    __syncwarp();
    if (e >= 0 && before == 0) base[e] += __popc(same);
    __syncwarp();
  }
}

}  // namespace laser
