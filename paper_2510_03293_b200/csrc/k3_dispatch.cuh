// K3: expert dispatch -- the stable grouping of pair ids t*k+j by expert -- together with the
// final slot order, expert ids and combine weights of every token.  One warp per group of 32
// tokens; the only atomics are warp-private shared-memory ORs.
//
// The ordered selection left, per group and expert, how many assignments of this call were
// made before the group (grp_base), and the call's offsets.  A token is assigned to an expert
// at most once, so a pair's position inside its expert's segment is
//     grp_base[group][e] + (tokens earlier in the group that were sent to e),
// which is also the load increment that token saw.  The warp first builds, per expert, the bit
// mask of its tokens sent there (the second term is then a population count), then every lane
// finishes its own token:
//   top-k branch (c* = 0): slots in score order.
//   c* > k: slots as the load-aware scan listed them (ascending load, then score rank); where
//           the scan left the choice as a bit mask over score ranks (the layer's mode word is
//           set), the slot order is rebuilt like that of c* == k.
//   c* == k: the set is the k best; slots ordered by (load seen, score rank), where the load
//            seen by rank j is L_in[e] + its position inside e's segment.
// w_j = s[expert of slot j], divided by the left-to-right sum over the slots if renormalising.
#pragma once
#include "laser_common.cuh"

namespace laser {

// Shared memory per warp: int32 base[E] | uint32 mask[E] | int32 pos[32*k] | int32 seen[32*k] |
// uint8 pe[32*k]; per block, in front of the warps' parts: int32 lin[E] | int32 off[E+1]
__host__ __device__ inline size_t k3_warp_smem_bytes(int E, int k) {
  return align256(2 * sizeof(int32_t) * (size_t)E + 2 * sizeof(int32_t) * 32 * (size_t)k +
                  32 * (size_t)k);
}
__host__ __device__ inline size_t k3_block_smem_bytes(int E) {
  return align256(sizeof(int32_t) * (2 * (size_t)E + 1));
}
__host__ __device__ inline int k3_warps_per_block(int E, int k) {
  const size_t per = k3_warp_smem_bytes(E, k);
  int w = (int)(((size_t)160 * 1024 - k3_block_smem_bytes(E)) / per);
  return w > 8 ? 8 : (w < 1 ? 1 : w);
}

// k3_group for k <= KR with a token's experts, positions and seen loads in registers (every loop
// over the k slots fully unrolled and guarded) instead of shared-memory arrays.
template <int KR>
__device__ __forceinline__ void k3_group_regs(const RouteArgs& A, int layer, int g,
                                              const int32_t* lin_s, const int32_t* off_s,
                                              unsigned char* mine) {
  const int lane = threadIdx.x & 31;
  const int k = A.k, c = A.c, E = A.E, T = A.T;
  int32_t* base = reinterpret_cast<int32_t*>(mine);
  uint32_t* mask = reinterpret_cast<uint32_t*>(base + E);

  const unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const long long t = (long long)g * 32 + lane;
  const bool valid = t < T;
  const int cs = valid ? reinterpret_cast<const uint16_t*>(ws + A.lay.cstar)[t] : 0;
  const uint8_t* cand = ws + A.lay.cand_ids + (size_t)t * c;
  const uint8_t* sel = ws + A.lay.sel_rank + (size_t)t * k;
  const int32_t* gb = reinterpret_cast<const int32_t*>(ws + A.lay.grp_base) + (size_t)g * E;
  const bool as_masks =
      reinterpret_cast<const int*>(ws + A.lay.ready)[mode_word_index(T)] != 0;

  // Everything a token can need is requested at once, whatever its branch turns out to be, so
  // that the group costs one round trip to memory: c*, the first KR ranked ids and scores, the
  // chosen ranks of a decision token, and per expert the group's base count and (E > 32) the
  // router's mask of the group's tokens without a decision.
  const float* sc = reinterpret_cast<const float*>(ws + A.lay.cand_scores) + (size_t)t * c;
  const bool have_fm = E > 32;
  const uint32_t* fmg = reinterpret_cast<const uint32_t*>(ws + A.lay.fmask) + (size_t)g * E;
  int idr[KR];
  float scr[KR];
  uint32_t chosen = 0;
#pragma unroll
  for (int j = 0; j < KR; ++j) { idr[j] = 0; scr[j] = 0.0f; }
  if (valid) {
    if (c == 8 && KR <= 8) {
      const uint2 v = *reinterpret_cast<const uint2*>(cand);
#pragma unroll
      for (int j = 0; j < KR; ++j) idr[j] = (int)(((j < 4 ? v.x : v.y) >> (8 * (j & 3))) & 255u);
    } else if (c == 4 && KR <= 4) {
      const uint32_t v = *reinterpret_cast<const uint32_t*>(cand);
#pragma unroll
      for (int j = 0; j < KR; ++j) idr[j] = (int)((v >> (8 * j)) & 255u);
    } else {
#pragma unroll
      for (int j = 0; j < KR; ++j)
        if (j < c) idr[j] = cand[j];
    }
    if (c % 4 == 0 && KR >= 4) {   // 16-byte aligned records: one or two full-width loads
      const float4 lo = *reinterpret_cast<const float4*>(sc);
      scr[0] = lo.x; scr[1] = lo.y; scr[2] = lo.z; scr[3] = lo.w;
      if constexpr (KR == 8) {
        if (c >= 8) {
          const float4 hi = *reinterpret_cast<const float4*>(sc + 4);
          scr[4] = hi.x; scr[5] = hi.y; scr[6] = hi.z; scr[7] = hi.w;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < KR; ++j)
        if (j < c) scr[j] = sc[j];
    }
    if (have_fm) chosen = reinterpret_cast<const uint32_t*>(ws + A.lay.sel_mask)[t];   // (used if as_masks)
  }
  for (int e = lane; e < E; e += 32) { base[e] = gb[e]; mask[e] = have_fm ? fmg[e] : 0u; }
  __syncwarp();
  int ex[KR], rk[KR];   // expert and candidate rank of slot j as the selection listed them
  float sr[KR];         // and its score
#pragma unroll
  for (int j = 0; j < KR; ++j) { ex[j] = idr[j]; rk[j] = j; sr[j] = scr[j]; }
  if (valid && cs > k) {   // a decision token: its ranks, experts and scores (few tokens)
#pragma unroll
    for (int j = 0; j < KR; ++j)
      if (j < k) {
        if (as_masks) { rk[j] = __ffs(chosen) - 1; chosen &= chosen - 1; }   // ascending rank
        else rk[j] = sel[j];
        ex[j] = cand[rk[j]];
        sr[j] = sc[rk[j]];
      }
  }
  if (valid && (!have_fm || cs > k)) {
#pragma unroll
    for (int j = 0; j < KR; ++j)
      if (j < k) atomicOr(&mask[ex[j]], 1u << lane);
  }
  __syncwarp();
  const unsigned below = (1u << lane) - 1;
  int pos[KR];
#pragma unroll
  for (int j = 0; j < KR; ++j)
    pos[j] = (valid && j < k) ? base[ex[j]] + __popc(mask[ex[j]] & below) : 0;

  int32_t* perm = A.perm + (size_t)layer * T * k;
  const int32_t pair0 = (int32_t)(t * k);
  float v[KR];     // weights in slot order
  int slot[KR];
#pragma unroll
  for (int j = 0; j < KR; ++j) { v[j] = sr[j]; slot[j] = j; }
  // top-k branch (c* = 0): score order, as ranked.  c* > k listed by the selection: as listed.
  if (valid && cs != 0 && !(cs > k && !as_masks)) {
    // the set is known, in ascending score rank (c* == k: the k best): slots by (load seen,
    // score rank); the load seen by the expert of rank j is L_in[e] + position
    // (relaxed variant: + the assignments made before the token's chunk instead)
    const int32_t* gb0 = nullptr;
    if (A.G != 1)
      gb0 = reinterpret_cast<const int32_t*>(ws + A.lay.grp_base) +
            (size_t)(A.G == 0 ? 0 : ((t / A.G) * A.G) / 32) * E;
    int32_t seen[KR];
#pragma unroll
    for (int j = 0; j < KR; ++j)
      seen[j] = j < k ? lin_s[ex[j]] + (gb0 ? gb0[ex[j]] : pos[j]) : 0;
#pragma unroll
    for (int j = 0; j < KR; ++j) {
      int sl = 0;
#pragma unroll
      for (int i = 0; i < KR; ++i)
        sl += (i < k && (seen[i] < seen[j] || (seen[i] == seen[j] && i < j))) ? 1 : 0;
      slot[j] = sl;
    }
#pragma unroll
    for (int s2 = 0; s2 < KR; ++s2) {
#pragma unroll
      for (int j = 0; j < KR; ++j)
        if (j < k && slot[j] == s2) v[s2] = sr[j];
    }
  }
  float sum = v[0];
#pragma unroll
  for (int j = 1; j < KR; ++j)
    if (j < k) sum = __fadd_rn(sum, v[j]);
  // ids and weights of the group's tokens are one contiguous block each: staged in shared
  // memory in slot order and written with full-width stores (the router's own copy of the
  // top-k branch's ids and weights is the same bits: its M_k is this left-to-right sum)
  int32_t* ids_s = base + 2 * E;
  float* w_s = reinterpret_cast<float*>(ids_s + 32 * k);
  if (valid) {
#pragma unroll
    for (int j = 0; j < KR; ++j)
      if (j < k) {
        ids_s[lane * k + slot[j]] = ex[j];
        w_s[lane * k + j] = A.renorm ? __fdiv_rn(v[j], sum) : v[j];
        perm[off_s[ex[j]] + pos[j]] = pair0 + slot[j];
      }
  }
  __syncwarp();
  const int n_out = (int)min(32LL, (long long)T - (long long)g * 32) * k;
  int32_t* ids = A.expert_ids + ((size_t)layer * T + (size_t)g * 32) * k;
  float* w = A.weights + ((size_t)layer * T + (size_t)g * 32) * k;
  for (int i = lane; i < n_out; i += 32) { ids[i] = ids_s[i]; w[i] = w_s[i]; }
}

// Group g (32 tokens) of absolute layer `layer`, by one warp.  lin_s / off_s: the layer's loads
// on entry and its offsets in shared memory; mine: k3_warp_smem_bytes() of scratch for the warp.
__device__ __forceinline__ void k3_group(const RouteArgs& A, int layer, int g,
                                         const int32_t* lin_s, const int32_t* off_s,
                                         unsigned char* mine) {
  if (A.k <= 8) {   // unrolled to the smallest of 2, 4, 8 slots that holds k
    if (A.k <= 2) k3_group_regs<2>(A, layer, g, lin_s, off_s, mine);
    else if (A.k <= 4) k3_group_regs<4>(A, layer, g, lin_s, off_s, mine);
    else k3_group_regs<8>(A, layer, g, lin_s, off_s, mine);
    return;
  }
  const int lane = threadIdx.x & 31;
  const int k = A.k, c = A.c, E = A.E, T = A.T;
  int32_t* base = reinterpret_cast<int32_t*>(mine);
  uint32_t* mask = reinterpret_cast<uint32_t*>(base + E);
  int32_t* pos = base + 2 * E;
  int32_t* seen = pos + 32 * k;
  uint8_t* pe = reinterpret_cast<uint8_t*>(seen + 32 * k);

  const unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const long long t = (long long)g * 32 + lane;
  const bool valid = t < T;
  const int cs = valid ? reinterpret_cast<const uint16_t*>(ws + A.lay.cstar)[t] : 0;
  const uint8_t* cand = ws + A.lay.cand_ids + (size_t)t * c;
  const uint8_t* sel = ws + A.lay.sel_rank + (size_t)t * k;
  const int32_t* gb = reinterpret_cast<const int32_t*>(ws + A.lay.grp_base) + (size_t)g * E;
  const bool as_masks =
      reinterpret_cast<const int*>(ws + A.lay.ready)[mode_word_index(T)] != 0;
  const uint32_t chosen = (valid && cs > k && as_masks)
                              ? reinterpret_cast<const uint32_t*>(ws + A.lay.sel_mask)[t] : 0u;
  // candidate rank of slot j as the selection left it (masks: ascending score rank)
  auto rank_of = [&](int j) -> int {
    if (cs <= k) return j;
    return as_masks ? (int)__fns(chosen, 0, j + 1) : (int)sel[j];
  };

  for (int e = lane; e < E; e += 32) { base[e] = gb[e]; mask[e] = 0; }
  __syncwarp();
  // mask[e]: which tokens of the group are sent to expert e.  A token is sent to an expert at
  // most once, so a pair's position inside its expert's segment is the group's base count plus
  // the number of earlier tokens of the group in that mask.
  if (valid)
    for (int j = 0; j < k; ++j) {
      const uint8_t e = cand[rank_of(j)];
      pe[lane * k + j] = e;
      atomicOr(&mask[e], 1u << lane);
    }
  __syncwarp();
  if (valid)
    for (int j = 0; j < k; ++j) {
      const int e = pe[lane * k + j];
      pos[lane * k + j] = base[e] + __popc(mask[e] & ((1u << lane) - 1));
    }
  if (!valid) return;

  const float* sc = reinterpret_cast<const float*>(ws + A.lay.cand_scores) + (size_t)t * c;
  const int32_t* off = off_s;
  int32_t* perm = A.perm + (size_t)layer * T * k;
  int32_t* ids = A.expert_ids + ((size_t)layer * T + t) * k;
  float* w = A.weights + ((size_t)layer * T + t) * k;
  const int32_t pair0 = (int32_t)(t * k);
  const int32_t* mypos = pos + lane * k;
  const uint8_t* mype = pe + lane * k;

  float sum = 0.0f;
  if (cs == 0) {   // top-k branch: score order, M_k = the left-to-right sum of the k best
    for (int j = 0; j < k; ++j) {
      const float v = sc[j];
      ids[j] = mype[j];
      w[j] = v;
      sum = j == 0 ? v : __fadd_rn(sum, v);
      perm[off[mype[j]] + mypos[j]] = pair0 + j;
    }
  } else if (cs > k && !as_masks) {
    for (int j = 0; j < k; ++j) {
      const int e = mype[j];
      ids[j] = e;
      const float v = sc[sel[j]];
      w[j] = v;
      sum = j == 0 ? v : __fadd_rn(sum, v);
      perm[off[e] + mypos[j]] = pair0 + j;
    }
  } else {
    // load seen by rank j: L_in[e] + position; L_in = L_out - count.  Smaller (load, j) first.
    // (Relaxed variant: the assignments made before the token's chunk take the position's place.)
    const int32_t* gb0 = nullptr;
    if (A.G != 1)
      gb0 = reinterpret_cast<const int32_t*>(ws + A.lay.grp_base) +
            (size_t)(A.G == 0 ? 0 : ((t / A.G) * A.G) / 32) * E;
    int32_t* myseen = seen + lane * k;
    for (int j = 0; j < k; ++j) {
      const int ej = mype[j];
      myseen[j] = lin_s[ej] + (gb0 ? gb0[ej] : mypos[j]);   // below 2^31: loads are int32
    }
    for (int j = 0; j < k; ++j) {
      const int ej = mype[j];
      const int32_t Lj = myseen[j];
      int slot = 0;
      for (int i = 0; i < k; ++i) {
        const int32_t Li = myseen[i];
        slot += (Li < Lj || (Li == Lj && i < j)) ? 1 : 0;
      }
      ids[slot] = ej;
      w[slot] = sc[rank_of(j)];
      perm[off[ej] + mypos[j]] = pair0 + slot;
    }
    if (A.renorm) {
      sum = w[0];
      for (int j = 1; j < k; ++j) sum = __fadd_rn(sum, w[j]);
    }
  }
  if (A.renorm)
    for (int j = 0; j < k; ++j) w[j] = __fdiv_rn(w[j], sum);
}

// (defined in one translation unit only: the one that launches it)
#ifdef LASER_DEFINE_K3_KERNEL
__global__ void __launch_bounds__(256, 5) k3_dispatch(const RouteArgs A) {
  extern __shared__ __align__(16) unsigned char k3_smem[];
  const int layer = A.layer0 + blockIdx.y;
  const int warp = threadIdx.x >> 5;
  const int warps = blockDim.x >> 5;
  const int g = blockIdx.x * warps + warp;
  const int E = A.E;
  // a layer whose selection gave up a wait has unwritten scratch records: leave it alone
  if (reinterpret_cast<const int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready)
          [abort_word_index(A.T)] != 0)
    return;

  // the layer's offsets and loads on entry (L_in = L_out - count), once per block
  int32_t* lin_s = reinterpret_cast<int32_t*>(k3_smem);
  int32_t* off_s = lin_s + E;
  {
    const int32_t* off_g = A.offsets + (size_t)layer * (E + 1);
    const int32_t* Lout = A.loads + (size_t)layer * E;
    for (int e = threadIdx.x; e <= E; e += blockDim.x) {
      off_s[e] = off_g[e];
      if (e < E) lin_s[e] = Lout[e] - (off_g[e + 1] - off_g[e]);
    }
  }
  __syncthreads();
  if (g >= A.lay.n_groups) return;
  k3_group(A, layer, g, lin_s, off_s,
           k3_smem + k3_block_smem_bytes(E) + (size_t)warp * k3_warp_smem_bytes(E, A.k));
}
#endif

}  // namespace laser
