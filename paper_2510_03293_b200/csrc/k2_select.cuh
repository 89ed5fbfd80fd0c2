// K2: the ordered, load-aware selection (Algorithm 1, StableSortByLoad + first k) and the
// per-token load update.  Tokens of one layer form one dependency chain, so one warp per
// layer walks them in row order with the load vector in shared memory; the other warps of
// the block only stage the next tile of candidate records.  Layers are independent blocks.
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK2Threads = 128;

__device__ __forceinline__ void k2_stage_tile(uint8_t* dst_ids, uint16_t* dst_cs,
                                              const uint8_t* src_ids, const uint16_t* src_cs,
                                              int ntok, int c, int tid, int nthreads) {
  const int bytes = ntok * c;
  const int n16 = bytes >> 4;
  const uint4* s4 = reinterpret_cast<const uint4*>(src_ids);
  uint4* d4 = reinterpret_cast<uint4*>(dst_ids);
  for (int i = tid; i < n16; i += nthreads) d4[i] = s4[i];
  for (int i = (n16 << 4) + tid; i < bytes; i += nthreads) dst_ids[i] = src_ids[i];
  for (int i = tid; i < ntok; i += nthreads) dst_cs[i] = src_cs[i];
}

// Adds one to a load counter; a counter at INT32_MAX stays there and raises the status bit.
__device__ __forceinline__ void bump_load(int32_t* L, int e, int32_t* status) {
  const int32_t v = L[e];
  if (v == 0x7fffffff) { if (status) atomicOr(status, 1); }
  else L[e] = v + 1;
}

// Dynamic shared memory: int32 L[E] | uint64 keys[c] | 2 x (uint8 ids[TILE*c], uint16 cs[TILE])
__global__ void __launch_bounds__(kK2Threads) k2_select(const RouteArgs A, int tile_tokens) {
  extern __shared__ __align__(16) unsigned char k2_smem[];
  const int layer = A.layer0 + blockIdx.x;
  const int T = A.T, E = A.E, k = A.k, c = A.c;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  int32_t* L = reinterpret_cast<int32_t*>(k2_smem);
  size_t off = align256(sizeof(int32_t) * E);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(k2_smem + off);
  off = align256(off + sizeof(unsigned long long) * c);
  const size_t ids_bytes = align256((size_t)tile_tokens * c);
  const size_t buf_bytes = ids_bytes + align256(sizeof(uint16_t) * tile_tokens);
  unsigned char* buf0 = k2_smem + off;

  unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const uint16_t* g_cs = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar);
  const uint8_t* g_ids = ws + A.lay.cand_ids;
  uint8_t* g_sel = ws + A.lay.sel_rank;
  int32_t* g_loads = A.loads + (size_t)layer * E;
  int32_t* g_eids = A.expert_ids + (size_t)layer * T * k;

  for (int e = tid; e < E; e += kK2Threads) L[e] = g_loads[e];
  const int n_tiles = (T + tile_tokens - 1) / tile_tokens;
  if (n_tiles > 0)
    k2_stage_tile(buf0, reinterpret_cast<uint16_t*>(buf0 + ids_bytes), g_ids, g_cs,
                  min(tile_tokens, T), c, tid, kK2Threads);
  __syncthreads();

  for (int tile = 0; tile < n_tiles; ++tile) {
    unsigned char* cur = buf0 + (size_t)(tile & 1) * buf_bytes;
    unsigned char* nxt = buf0 + (size_t)((tile + 1) & 1) * buf_bytes;
    const int t0 = tile * tile_tokens;
    const int ntok = min(tile_tokens, T - t0);
    if (warp > 0) {
      if (tile + 1 < n_tiles) {
        const int t1 = t0 + tile_tokens;
        k2_stage_tile(nxt, reinterpret_cast<uint16_t*>(nxt + ids_bytes), g_ids + (size_t)t1 * c,
                      g_cs + t1, min(tile_tokens, T - t1), c, tid - 32, kK2Threads - 32);
      }
    } else {
      const uint8_t* s_ids = cur;
      const uint16_t* s_cs = reinterpret_cast<const uint16_t*>(cur + ids_bytes);
      for (int i = 0; i < ntok; ++i) {
        const int cs = s_cs[i];
        const uint8_t* ids = s_ids + (size_t)i * c;
        const size_t t = (size_t)(t0 + i);
        if (cs == 0) {
          // top-k branch: the choice is already written; only the loads move
          for (int j = lane; j < k; j += 32) bump_load(L, ids[j], A.status);
        } else if (cs <= 32) {
          // one candidate per lane; key = (load, score rank); rank by counting smaller keys
          const int e = lane < cs ? ids[lane] : 0;
          const unsigned long long key =
              lane < cs ? (((unsigned long long)(uint32_t)L[e]) << 8) | (unsigned)lane : ~0ull;
          int cnt = 0;
          for (int j = 0; j < cs; ++j) cnt += (__shfl_sync(0xffffffffu, key, j) < key) ? 1 : 0;
          if (lane < cs && cnt < k) {
            g_eids[t * k + cnt] = e;
            g_sel[t * k + cnt] = (uint8_t)lane;
            bump_load(L, e, A.status);
          }
        } else {
          // wide candidate sets: keys through shared memory, several candidates per lane
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
              g_eids[t * k + cnt] = ids[j];
              g_sel[t * k + cnt] = (uint8_t)j;
              chosen |= 1u << it;
            }
          }
          // loads move only after every lane has finished reading the keys
          __syncwarp();
          it = 0;
          for (int j = lane; j < cs; j += 32, ++it)
            if ((chosen >> it) & 1u) bump_load(L, ids[j], A.status);
        }
        __syncwarp();
      }
    }
    __syncthreads();
  }
  for (int e = tid; e < E; e += kK2Threads) g_loads[e] = L[e];
}

// Combine weights of tokens routed by the load-aware branch: w_j = s[chosen_j], divided by
// their left-to-right sum when renormalising.  One thread per token.
__global__ void k2_weights(const RouteArgs A) {
  const int layer = A.layer0 + blockIdx.y;
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= A.T) return;
  unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  if (reinterpret_cast<const uint16_t*>(ws + A.lay.cstar)[t] == 0) return;
  const float* sc = reinterpret_cast<const float*>(ws + A.lay.cand_scores) + (size_t)t * A.c;
  const uint8_t* sel = ws + A.lay.sel_rank + (size_t)t * A.k;
  float* w = A.weights + ((size_t)layer * A.T + t) * A.k;
  float sum = 0.0f;
  for (int j = 0; j < A.k; ++j) {
    const float v = sc[sel[j]];
    w[j] = v;
    sum = j == 0 ? v : __fadd_rn(sum, v);
  }
  if (A.renorm)
    for (int j = 0; j < A.k; ++j) w[j] = __fdiv_rn(w[j], sum);
}

}  // namespace laser
