// K2: the ordered, load-aware selection (Algorithm 1, StableSortByLoad + first k) and the
// per-token load update.  Tokens of one layer form one dependency chain; layers are
// independent thread blocks.
//
// Only tokens whose candidate set is larger than k (c* > k, "decision tokens") have a
// load-dependent choice.  Every other token (top-k branch, or c* == k) sends its k best
// experts whatever the loads are, so its increments are known without the chain.  The block
// therefore splits the work:
//   prep warps   stage a tile of candidate records in shared memory and, per group of 32
//                tokens, count the fixed increments per expert (group totals) and, for every
//                candidate of every decision token, the fixed increments of earlier tokens
//                of the same group (ballot + popcount);
//   chain warp   walks the decision tokens only: load seen by candidate j =
//                L[e_j] (all earlier groups + earlier decisions) + its in-group prefix;
//                ranks the candidates by (load, score rank) with warp shuffles, bumps the
//                k winners, and adds the group totals at each group end.
// The slot order of c* == k tokens, which depends on the loads they saw, is reconstructed
// afterwards from the dispatch ranks (k3_finalize).
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK2Threads = 256;
constexpr int kK2PrepWarps = kK2Threads / 32 - 1;
constexpr int kK2Tile = 256;             // tokens per shared-memory buffer
constexpr int kK2Groups = kK2Tile / 32;
constexpr int kK2FastMaxLoad = 1 << 26;  // 32-bit keys (load << 5 | rank) need loads below this

struct K2Buffers {
  uint8_t* ids;     // [kK2Tile * c] ranked candidate ids
  uint8_t* pre;     // [kK2Tile * c] in-group fixed increments seen by each candidate
  uint16_t* cs;     // [kK2Tile]
  int32_t* gtot;    // [kK2Groups * E] fixed increments per group and expert
};

__host__ __device__ inline size_t k2_buffer_bytes(int E, int c) {
  return 2 * align256((size_t)kK2Tile * c) + align256(sizeof(uint16_t) * kK2Tile) +
         align256(sizeof(int32_t) * kK2Groups * E);
}

__device__ __forceinline__ K2Buffers k2_carve(unsigned char* base, int E, int c) {
  K2Buffers b;
  b.ids = base;
  b.pre = base + align256((size_t)kK2Tile * c);
  b.cs = reinterpret_cast<uint16_t*>(base + 2 * align256((size_t)kK2Tile * c));
  b.gtot = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(b.cs) +
                                      align256(sizeof(uint16_t) * kK2Tile));
  return b;
}

// Prepares one group of 32 tokens (lane = token) of a tile.
__device__ __forceinline__ void k2_prep_group(const K2Buffers& b, int g, int ntok,
                                              const uint8_t* g_ids, const uint16_t* g_cs, int E,
                                              int k, int c, int lane) {
  const int tok = g * 32 + lane;
  const bool valid = tok < ntok;
  const int n_here = min(32, ntok - g * 32);
  // stage this group's records
  {
    const int bytes = n_here * c;
    const uint8_t* src = g_ids + (size_t)g * 32 * c;
    uint8_t* dst = b.ids + (size_t)g * 32 * c;
    const int n16 = bytes >> 4;
    for (int i = lane; i < n16; i += 32)
      reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
    for (int i = (n16 << 4) + lane; i < bytes; i += 32) dst[i] = src[i];
  }
  const int cs = valid ? g_cs[tok] : 0;
  b.cs[tok] = (uint16_t)cs;
  int32_t* gt = b.gtot + g * E;
  for (int e = lane; e < E; e += 32) gt[e] = 0;
  __syncwarp();
  const bool fixed = valid && cs <= k;
  const uint8_t* my = b.ids + (size_t)tok * c;
  if (fixed)
    for (int j = 0; j < k; ++j) atomicAdd(&gt[my[j]], 1);
  unsigned dmask = __ballot_sync(0xffffffffu, valid && cs > k);
  while (dmask) {
    const int dl = __ffs(dmask) - 1;
    dmask &= dmask - 1;
    const int csd = __shfl_sync(0xffffffffu, cs, dl);
    const uint8_t* cand = b.ids + (size_t)(g * 32 + dl) * c;
    const unsigned before = (1u << dl) - 1;
    int mine = 0;
    for (int r = 0; r < csd; ++r) {
      const int e = cand[r];
      bool hit = false;
      if (fixed)
        for (int j = 0; j < k; ++j) hit |= (my[j] == e);
      const int cnt = __popc(__ballot_sync(0xffffffffu, hit) & before);
      if (lane == (r & 31)) mine = cnt;
      if ((r & 31) == 31 || r == csd - 1) {
        const int rr = (r & ~31) + lane;
        if (rr <= r) b.pre[(size_t)(g * 32 + dl) * c + rr] = (uint8_t)mine;
      }
    }
  }
}

// Chain over one tile, candidate sets no wider than a warp, loads below 2^26.
template <int CMAX>
__device__ __forceinline__ void k2_chain_tile(int32_t* L, const K2Buffers& b, int ntok, int E,
                                              int k, int c, uint8_t* g_sel, int lane) {
  const int n_groups = (ntok + 31) >> 5;
  for (int g = 0; g < n_groups; ++g) {
    const int tok = g * 32 + lane;
    const int cs_l = tok < ntok ? b.cs[tok] : 0;
    unsigned dmask = __ballot_sync(0xffffffffu, cs_l > k);
    while (dmask) {
      const int dl = __ffs(dmask) - 1;
      dmask &= dmask - 1;
      const int csd = __shfl_sync(0xffffffffu, cs_l, dl);
      const size_t td = (size_t)(g * 32 + dl);
      const bool mine = lane < csd;
      const int id = mine ? b.ids[td * c + lane] : 0;
      const int p = mine ? b.pre[td * c + lane] : 0;
      const int32_t Lraw = mine ? L[id] : 0;
      const uint32_t key = mine ? (((uint32_t)(Lraw + p) << 5) | (uint32_t)lane) : 0xffffffffu;
      int cnt = 0;
#pragma unroll
      for (int j = 0; j < CMAX; ++j) {
        const uint32_t other = __shfl_sync(0xffffffffu, key, j);
        if (j < csd) cnt += other < key ? 1 : 0;
      }
      if (mine && cnt < k) {
        L[id] = Lraw + 1;
        g_sel[td * k + cnt] = (uint8_t)lane;
      }
      __syncwarp();
    }
    const int32_t* gt = b.gtot + g * E;
    for (int e = lane; e < E; e += 32) L[e] += gt[e];
    __syncwarp();
  }
}

// Fallback for candidate sets or k wider than a warp, or loads of 2^26 and more: one warp
// walks every token of the range; 64-bit keys (load, score rank) go through shared memory.
__device__ __forceinline__ void k2_chain_wide(int32_t* L, unsigned long long* keys,
                                              const uint16_t* g_cs, const uint8_t* g_ids,
                                              uint8_t* g_sel, int ntot, int k, int c, int lane) {
  for (long long t = 0; t < ntot; ++t) {
    const int cs = g_cs[t];
    const uint8_t* ids = g_ids + t * c;
    if (cs <= k) {
      for (int j = lane; j < k; j += 32) L[ids[j]] += 1;
    } else {
      for (int j = lane; j < cs; j += 32)
        keys[j] = (((unsigned long long)(uint32_t)L[ids[j]]) << 8) | (unsigned)j;
      __syncwarp();
      unsigned chosen = 0;
      int it = 0;
      for (int j = lane; j < cs; j += 32, ++it) {
        const unsigned long long key = keys[j];
        int cnt = 0;
        for (int i2 = 0; i2 < cs; ++i2) cnt += (keys[i2] < key) ? 1 : 0;
        if (cnt < k) {
          g_sel[t * k + cnt] = (uint8_t)j;
          chosen |= 1u << it;
        }
      }
      __syncwarp();  // loads move only after every lane has finished reading the keys
      it = 0;
      for (int j = lane; j < cs; j += 32, ++it)
        if ((chosen >> it) & 1u) L[ids[j]] += 1;
    }
    __syncwarp();
  }
}

// Dynamic shared memory: int32 L[E] | uint64 keys[c] | 2 x K2Buffers
__global__ void __launch_bounds__(kK2Threads) k2_select(const RouteArgs A) {
  extern __shared__ __align__(16) unsigned char k2_smem[];
  const int layer = A.layer0 + blockIdx.x;
  const int E = A.E, k = A.k, c = A.c;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tb = A.tok_begin, ntot = A.tok_end - A.tok_begin;

  int32_t* L = reinterpret_cast<int32_t*>(k2_smem);
  unsigned long long* keys =
      reinterpret_cast<unsigned long long*>(k2_smem + align256(sizeof(int32_t) * E));
  unsigned char* buf0 = reinterpret_cast<unsigned char*>(keys) +
                        align256(sizeof(unsigned long long) * c);
  const size_t buf_bytes = k2_buffer_bytes(E, c);

  unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const uint16_t* g_cs = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar) + tb;
  const uint8_t* g_ids = ws + A.lay.cand_ids + (size_t)tb * c;
  uint8_t* g_sel = ws + A.lay.sel_rank + (size_t)tb * k;
  int32_t* g_loads = A.loads + (size_t)layer * E;

  int too_big = 0;
  for (int e = tid; e < E; e += kK2Threads) {
    const int32_t v = g_loads[e];
    L[e] = v;
    // a counter within T of 2^31-1 could wrap during the call: raise the status bit
    if (v < 0 || v > 0x7fffffff - A.T) { if (A.status) atomicOr(A.status, 1); }
    if (v < 0 || v > kK2FastMaxLoad - A.T) too_big = 1;
  }
  if (__syncthreads_or(too_big) || c > 32 || k > 32) {
    if (warp == 0) {
      k2_chain_wide(L, keys, g_cs, g_ids, g_sel, ntot, k, c, lane);
      for (int e = lane; e < E; e += 32) g_loads[e] = L[e];
    }
    return;
  }
  const int n_tiles = (ntot + kK2Tile - 1) / kK2Tile;

  auto prep_tile = [&](int tile, int first_warp, int n_warps) {
    const K2Buffers b = k2_carve(buf0 + (size_t)(tile & 1) * buf_bytes, E, c);
    const int t0 = tile * kK2Tile;
    const int ntok = min(kK2Tile, ntot - t0);
    const int n_groups = (ntok + 31) >> 5;
    for (int g = warp - first_warp; g < n_groups; g += n_warps)
      k2_prep_group(b, g, ntok, g_ids + (size_t)t0 * c, g_cs + t0, E, k, c, lane);
  };

  if (n_tiles > 0) prep_tile(0, 0, kK2Threads / 32);
  __syncthreads();
  for (int tile = 0; tile < n_tiles; ++tile) {
    if (warp > 0) {
      if (tile + 1 < n_tiles) prep_tile(tile + 1, 1, kK2PrepWarps);
    } else {
      const K2Buffers b = k2_carve(buf0 + (size_t)(tile & 1) * buf_bytes, E, c);
      const int t0 = tile * kK2Tile;
      const int ntok = min(kK2Tile, ntot - t0);
      uint8_t* sel = g_sel + (size_t)t0 * k;
      if (c <= 4) k2_chain_tile<4>(L, b, ntok, E, k, c, sel, lane);
      else if (c <= 8) k2_chain_tile<8>(L, b, ntok, E, k, c, sel, lane);
      else if (c <= 16) k2_chain_tile<16>(L, b, ntok, E, k, c, sel, lane);
      else k2_chain_tile<32>(L, b, ntok, E, k, c, sel, lane);
    }
    __syncthreads();
  }
  for (int e = tid; e < E; e += kK2Threads) g_loads[e] = L[e];
}

}  // namespace laser
