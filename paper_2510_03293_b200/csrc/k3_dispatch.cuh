// K3: expert dispatch from the chosen experts -- per-call counts, exclusive offsets, the
// stable grouping of pair ids t*k+j by expert -- and device-bin load sums (N_g = sum of the
// counts of the experts placed on bin g).  Four passes, none of which uses an atomic:
//   k3_hist     block histograms from warp-private counters (match-any + leader add)
//   k3_scan     per-expert prefix over blocks, warp-scan prefix over experts, bin sums
//   k3_rank     stable destination index of every pair with warp-private running bases
//   k3_finalize per token: final slot order, expert ids, combine weights, perm entries
// A token is assigned to an expert at most once, so a pair's position inside its expert's
// segment is the number of earlier tokens sent to that expert -- which is also the load
// increment that token saw.  k3_finalize uses this to order the slots of tokens whose set
// was fixed (c* == k) but whose listing order is by (load seen, score rank).
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK3Threads = 256;
constexpr int kK3Warps = kK3Threads / 32;
constexpr int kK3PairsPerWarp = kDispatchPairsPerBlock / kK3Warps;

// Counts the experts of this warp's contiguous span of pair ids into hist (warp-private).
struct PairSource {
  const uint16_t* cstar;
  const uint8_t* cand_ids;
  const uint8_t* sel_rank;
  int k, c;
  __device__ __forceinline__ int expert(long long p) const {
    const long long t = p / k;
    const int j = (int)(p - t * k);
    return cand_ids[t * c + pair_rank(cstar, sel_rank, k, t, j)];
  }
};

__device__ __forceinline__ PairSource pair_source(const RouteArgs& A, int layer) {
  const unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  PairSource s;
  s.cstar = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar);
  s.cand_ids = ws + A.lay.cand_ids;
  s.sel_rank = ws + A.lay.sel_rank;
  s.k = A.k; s.c = A.c;
  return s;
}

__device__ __forceinline__ void k3_warp_hist(const PairSource& src, long long begin,
                                             long long end, int32_t* hist, int lane) {
  for (long long p0 = begin; p0 < end; p0 += 32) {
    const long long p = p0 + lane;
    const int e = p < end ? src.expert(p) : -1;
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
  const PairSource src = pair_source(A, layer);
  for (int i = tid; i < kK3Warps * E; i += kK3Threads) k3_smem[i] = 0;
  __syncthreads();
  const long long begin = min(n, (long long)blockIdx.x * kDispatchPairsPerBlock +
                                     (long long)warp * kK3PairsPerWarp);
  const long long end = min(n, begin + kK3PairsPerWarp);
  k3_warp_hist(src, begin, end, k3_smem + warp * E, lane);
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

__global__ void __launch_bounds__(kK3Threads) k3_rank(const RouteArgs A) {
  extern __shared__ int32_t k3_smem[];  // [kK3Warps][E] histograms, then running bases
  const int layer = A.layer0 + blockIdx.y;
  const int E = A.E, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long n = (long long)A.T * A.k;
  const PairSource src = pair_source(A, layer);
  int32_t* pair_dst = reinterpret_cast<int32_t*>(A.ws + (size_t)layer * A.ws_ls + A.lay.pair_dst);
  for (int i = tid; i < kK3Warps * E; i += kK3Threads) k3_smem[i] = 0;
  __syncthreads();
  const long long begin = min(n, (long long)blockIdx.x * kDispatchPairsPerBlock +
                                     (long long)warp * kK3PairsPerWarp);
  const long long end = min(n, begin + kK3PairsPerWarp);
  k3_warp_hist(src, begin, end, k3_smem + warp * E, lane);
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
    const int e = p < end ? src.expert(p) : -1;
    const unsigned same = __match_any_sync(0xffffffffu, e);
    const unsigned before = same & ((1u << lane) - 1);
    if (e >= 0) pair_dst[p] = base[e] + __popc(before);
    __syncwarp();
    if (e >= 0 && before == 0) base[e] += __popc(same);
    __syncwarp();
  }
}

// One thread per token: final slot order, expert ids, combine weights and perm entries.
//   top-k branch (c* = 0): slots in score order; ids and weights were written by the router.
//   c* > k: slots as the load-aware scan listed them (ascending load, then score rank).
//   c* == k: the set is the k best; slots ordered by (load seen, score rank), where the load
//            seen by slot j is L_in[e] + (position of the pair inside e's segment).
// w_j = s[expert of slot j], divided by the left-to-right sum over the slots if renormalising.
__global__ void k3_finalize(const RouteArgs A) {
  const int layer = A.layer0 + blockIdx.y;
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= A.T) return;
  const int k = A.k, c = A.c, E = A.E;
  const unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const int cs = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar)[t];
  const uint8_t* cand = ws + A.lay.cand_ids + (size_t)t * c;
  const float* sc = reinterpret_cast<const float*>(ws + A.lay.cand_scores) + (size_t)t * c;
  const uint8_t* sel = ws + A.lay.sel_rank + (size_t)t * k;
  const int32_t* dst = reinterpret_cast<const int32_t*>(ws + A.lay.pair_dst) + (size_t)t * k;
  int32_t* perm = A.perm + (size_t)layer * A.T * k;
  int32_t* ids = A.expert_ids + ((size_t)layer * A.T + t) * k;
  float* w = A.weights + ((size_t)layer * A.T + t) * k;
  const int32_t pair0 = (int32_t)(t * k);

  if (cs == 0) {
    for (int j = 0; j < k; ++j) perm[dst[j]] = pair0 + j;
    return;
  }
  float sum = 0.0f;
  if (cs > k) {
    for (int j = 0; j < k; ++j) {
      const int r = sel[j];
      ids[j] = cand[r];
      const float v = sc[r];
      w[j] = v;
      sum = j == 0 ? v : __fadd_rn(sum, v);
      perm[dst[j]] = pair0 + j;
    }
  } else {
    // load seen by rank j: L_out[e] - count[e] + (dst - offsets[e]); smaller (load, j) first
    const int32_t* off = A.offsets + (size_t)layer * (E + 1);
    const int32_t* Lout = A.loads + (size_t)layer * E;
    for (int j = 0; j < k; ++j) {
      const int ej = cand[j];
      const long long Lj = (long long)Lout[ej] - off[ej + 1] + dst[j];
      int slot = 0;
      for (int i = 0; i < k; ++i) {
        const int ei = cand[i];
        const long long Li = (long long)Lout[ei] - off[ei + 1] + dst[i];
        slot += (Li < Lj || (Li == Lj && i < j)) ? 1 : 0;
      }
      ids[slot] = ej;
      w[slot] = sc[j];
      perm[dst[j]] = pair0 + slot;
    }
    if (A.renorm) {
      sum = w[0];
      for (int j = 1; j < k; ++j) sum = __fadd_rn(sum, w[j]);
    }
  }
  if (A.renorm)
    for (int j = 0; j < k; ++j) w[j] = __fdiv_rn(w[j], sum);
}

}  // namespace laser
