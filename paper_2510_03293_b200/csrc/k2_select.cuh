// K2: the ordered, load-aware selection (Algorithm 1, StableSortByLoad + first k) and the
// per-token load update.  Tokens of one layer form one dependency chain; layers are
// independent thread blocks.
//
// Only tokens whose candidate set is larger than k (c* > k, "decision tokens") have a
// load-dependent choice.  Every other token (top-k branch, or c* == k) sends its k best
// experts whatever the loads are, so its increments are known without the chain.  The block
// therefore splits the work, tile by tile (double buffered in shared memory):
//   prep warps   stage the candidate records (cp.async), count the fixed increments per group
//                of 32 tokens, prefix them over the tile, and write a dense, ordered list of
//                the tile's decision tokens.  A list entry holds one word per lane of the
//                chain warp with the addend (fixed increments seen so far in the tile << 5 |
//                score rank), so that a candidate's key is
//                    (load at tile start + decisions so far) << 5 + addend.
//   chain warp   walks the list with the next entry prefetched into registers; per entry it
//                forms the keys, ranks each candidate by counting smaller keys (one shuffle
//                per candidate), bumps the k winners and records their score ranks.
// A single warp is a slow sequential machine (a dependent instruction issues every few
// cycles), so everything that does not depend on the loads is moved into the prep warps and
// the chain loop is kept to a few dozen instructions.
// Two chain layouts:
//   E <= 32, c <= 16   lane = expert, loads stay in a register of the chain warp;
//   otherwise          lane = candidate, loads in shared memory.
// The slot order of c* == k tokens, which depends on the loads they saw, is reconstructed
// afterwards from the dispatch ranks (k3_finalize).
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kK2Threads = 256;
constexpr int kK2Warps = kK2Threads / 32;
constexpr int kK2Tile = 256;             // tokens per shared-memory buffer
constexpr int kK2Groups = kK2Tile / 32;
constexpr int kK2FastMaxLoad = 1 << 25;  // 32-bit keys (load << 5 | rank) stay below 2^31
constexpr uint32_t kK2NoCand = 0x80000000u;
constexpr long long kK2WaitCycles = 4000000000LL;  // give up waiting for the router after ~2 s

// A list entry is LW lane words, then 4 words of shuffle source lanes, then the sel base.
__host__ __device__ inline int k2_lane_words(int E, int c) {
  return (E <= 32 && c <= 16) ? ((E + 7) & ~7) : ((c + 3) & ~3);
}
__host__ __device__ inline int k2_entry_words(int E, int c) { return k2_lane_words(E, c) + 8; }

struct K2Buffers {
  uint8_t* ids;     // [kK2Tile * c]      staged ranked candidate ids
  uint16_t* cs;     // [kK2Tile]          staged c*
  uint32_t* gB;     // [kK2Groups * 32]   E <= 32: per group and expert, ballot of fixed senders
  int32_t* gtot;    // [kK2Groups * max(E,32)] fixed increments per group and expert, then their
                    //                    exclusive prefix over the groups of the tile
  int32_t* ttot;    // [max(E,32)]        fixed increments of the whole tile per expert
  int32_t* dcount;  // [kK2Groups]        decision tokens per group
  uint32_t* list;   // [(kK2Tile + 1) * entry words] decision-token entries
};

__host__ __device__ inline size_t k2_buffer_bytes(int E, int c) {
  const int Ew = E > 32 ? E : 32;
  return align256((size_t)kK2Tile * c) + align256(sizeof(uint16_t) * kK2Tile) +
         align256(sizeof(uint32_t) * kK2Groups * 32) + align256(sizeof(int32_t) * kK2Groups * Ew) +
         align256(sizeof(int32_t) * Ew) + align256(sizeof(int32_t) * kK2Groups) +
         align256(sizeof(uint32_t) * (kK2Tile + 1) * k2_entry_words(E, c));
}

// Shared memory of the selection role: int32 L[E] | uint64 keys[c] | 2 x K2Buffers; the wide
// fallback (c or k above 32) needs only the first two.
__host__ __device__ inline size_t k2_smem_bytes(int E, int c, int k) {
  const size_t base = align256(sizeof(int32_t) * E) + align256(sizeof(unsigned long long) * c);
  if (c > 32 || k > 32) return base;
  return base + 2 * k2_buffer_bytes(E, c);
}

__device__ __forceinline__ K2Buffers k2_carve(unsigned char* p, int E, int c) {
  const int Ew = E > 32 ? E : 32;
  K2Buffers b;
  b.ids = p;                                 p += align256((size_t)kK2Tile * c);
  b.cs = reinterpret_cast<uint16_t*>(p);     p += align256(sizeof(uint16_t) * kK2Tile);
  b.gB = reinterpret_cast<uint32_t*>(p);     p += align256(sizeof(uint32_t) * kK2Groups * 32);
  b.gtot = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * kK2Groups * Ew);
  b.ttot = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * Ew);
  b.dcount = reinterpret_cast<int32_t*>(p);  p += align256(sizeof(int32_t) * kK2Groups);
  b.list = reinterpret_cast<uint32_t*>(p);
  return b;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_all;" ::: "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Waits until the router blocks that produce tokens [t_first, t_last] of this layer have
// published their records.  Bounded: gives up after kK2WaitCycles and returns false.
__device__ __forceinline__ bool k2_wait_ready(const int* ready, int router_rows, int t_first,
                                              int t_last) {
  const long long start = clock64();
  for (int rt = t_first / router_rows; rt <= t_last / router_rows; ++rt) {
    while (ld_acquire(ready + rt) == 0) {
      if (clock64() - start > kK2WaitCycles) return false;
      __nanosleep(200);
    }
  }
  return true;
}

// Issues the copies of one group's records (32 tokens) into the tile buffer.
__device__ __forceinline__ void k2_stage_group(const K2Buffers& b, int g, int ntok,
                                               const uint8_t* g_ids, const uint16_t* g_cs, int c,
                                               int lane) {
  const int n_here = min(32, ntok - g * 32);
  const uint8_t* src = g_ids + (size_t)g * 32 * c;
  uint8_t* dst = b.ids + g * 32 * c;
  if (n_here == 32) {
    for (int i = lane; i < 2 * c; i += 32) cp_async16(dst + 16 * i, src + 16 * i);
    if (lane < 4) cp_async16(b.cs + g * 32 + lane * 8, g_cs + g * 32 + lane * 8);
  } else {
    for (int i = lane; i < n_here * c; i += 32) dst[i] = __ldcg(src + i);
    b.cs[g * 32 + lane] = lane < n_here ? __ldcg(g_cs + g * 32 + lane) : (uint16_t)0;
  }
}

// Phase 1 for one staged group (lane = token): decision count and the fixed increments.
__device__ __forceinline__ void k2_count_group(const K2Buffers& b, int g, int ntok, int E, int Ew,
                                               int k, int c, bool small_e, int lane) {
  const int tok = g * 32 + lane;
  const bool valid = tok < ntok;
  const int cs = valid ? b.cs[tok] : 0;
  const bool fixed = valid && cs <= k;
  const uint8_t* my = b.ids + tok * c;
  const unsigned dmask = __ballot_sync(0xffffffffu, valid && cs > k);
  if (lane == 0) b.dcount[g] = __popc(dmask);
  if (small_e) {
    uint32_t m = 0;
    if (fixed)
      for (int j = 0; j < k; ++j) m |= 1u << my[j];
    uint32_t mineB = 0;
    for (int e = 0; e < E; ++e) {
      const uint32_t B = __ballot_sync(0xffffffffu, (m >> e) & 1u);
      if (lane == e) mineB = B;
    }
    b.gB[g * 32 + lane] = mineB;
  } else {
    int32_t* gt = b.gtot + g * Ew;
    for (int e = lane; e < E; e += 32) gt[e] = 0;
    __syncwarp();
    if (fixed)
      for (int j = 0; j < k; ++j) atomicAdd(&gt[my[j]], 1);
  }
}

// Phase 2 for one group: appends its decision tokens to the tile's list.
// LW lane words per entry, EW words per entry.
template <int KREG>
__device__ __forceinline__ void k2_list_group(const K2Buffers& b, int g, int ntok, int E, int Ew,
                                              int k, int c, bool small_e, int LW, int EW,
                                              int lane) {
  const int tok = g * 32 + lane;
  const bool valid = tok < ntok;
  const int cs = valid ? b.cs[tok] : 0;
  const uint8_t* my = b.ids + tok * c;
  const bool dec = valid && cs > k;
  const unsigned dmask = __ballot_sync(0xffffffffu, dec);
  if (dmask == 0) return;
  int dbase = 0;
  for (int g2 = 0; g2 < g; ++g2) dbase += b.dcount[g2];
  const int nd = __popc(dmask);
  const unsigned below = (1u << lane) - 1;
  const int32_t* gpre = b.gtot + g * Ew;   // fixed increments in earlier groups of the tile

  if (small_e) {
    // lane = decision token builds its own entry (lane words indexed by expert)
    uint32_t* ent0 = b.list + dbase * EW;
    for (int i = lane; i < nd * LW; i += 32) ent0[(i / LW) * EW + (i % LW)] = kK2NoCand;
    __syncwarp();
    if (dec) {
      uint32_t* ent = ent0 + __popc(dmask & below) * EW;
      const uint32_t* B = b.gB + g * 32;
      uint32_t cmask = 0;
      for (int r = 0; r < cs; ++r) {
        const int e = my[r];
        cmask |= 1u << e;
        ent[e] = ((uint32_t)(gpre[e] + __popc(B[e] & below)) << 5) | (uint32_t)r;
      }
      // unused shuffle sources point at a lane that holds no candidate
      const uint32_t pad = E < 32 ? 31u : (uint32_t)(__ffs(~cmask) - 1);
      uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t v = j < cs ? (uint32_t)my[j] : pad;
        w[j >> 2] |= v << (8 * (j & 3));
      }
      ent[LW] = w[0]; ent[LW + 1] = w[1]; ent[LW + 2] = w[2]; ent[LW + 3] = w[3];
      ent[LW + 4] = (uint32_t)(tok * k);
    }
    return;
  }

  // lane = candidate: one decision token after the other, one ballot per candidate
  const bool fixed = valid && cs <= k;
  int myid[KREG > 0 ? KREG : 1];
#pragma unroll
  for (int j = 0; j < KREG; ++j) myid[j] = (fixed && j < k) ? my[j] : -1;
  unsigned rest = dmask;
  while (rest) {
    const int dl = __ffs(rest) - 1;
    rest &= rest - 1;
    const unsigned before = (1u << dl) - 1;
    uint32_t* ent = b.list + (dbase + __popc(dmask & before)) * EW;
    const int csd = __shfl_sync(0xffffffffu, cs, dl);
    const uint8_t* cand = b.ids + (g * 32 + dl) * c;
    int mine = 0;
    for (int r = 0; r < csd; ++r) {   // csd <= 32 on this path
      const int e = cand[r];
      bool hit = false;
      if (KREG > 0) {
#pragma unroll
        for (int j = 0; j < KREG; ++j) hit |= (myid[j] == e);
      } else if (fixed) {
        for (int j = 0; j < k; ++j) hit |= (my[j] == e);
      }
      const int cnt = __popc(__ballot_sync(0xffffffffu, hit) & before);
      if (lane == r) mine = cnt;
    }
    uint32_t word = 0x8000u;
    if (lane < csd) {
      const int e = cand[lane];
      word = ((uint32_t)(mine + gpre[e]) << 5) | (uint32_t)lane | ((uint32_t)e << 16);
    }
    if (lane < LW) ent[lane] = word;
    if (lane == 0) ent[LW + 4] = (uint32_t)((g * 32 + dl) * k);
  }
}

// Chain over one tile's list, lane = expert.  Le32 = (load of expert `lane`) << 5.
template <int CMAX>
__device__ __forceinline__ void k2_chain_experts(uint32_t& Le32, const uint32_t* list, int n_dec,
                                                 int k, int LW, int EW, uint8_t* sel, int lane) {
  constexpr int SW = (CMAX + 3) / 4;
  const bool has = lane < LW;
  uint32_t add_n = has ? list[lane] : kK2NoCand, base_n = list[LW + 4];
  uint32_t src_n[SW];
#pragma unroll
  for (int q = 0; q < SW; ++q) src_n[q] = list[LW + q];
#pragma unroll 1
  for (int i = 0; i < n_dec; ++i) {
    const uint32_t add = add_n, base = base_n;
    uint32_t src[SW];
#pragma unroll
    for (int q = 0; q < SW; ++q) src[q] = src_n[q];
    const uint32_t* nx = list + (i + 1) * EW;   // the list has one spare entry
    if (has) add_n = nx[lane];
    base_n = nx[LW + 4];
#pragma unroll
    for (int q = 0; q < SW; ++q) src_n[q] = nx[LW + q];
    const uint32_t key = Le32 + add;
    // all shuffles are issued before the first compare, so their latencies overlap
    uint32_t other[CMAX];
#pragma unroll
    for (int j = 0; j < CMAX; ++j)
      other[j] = __shfl_sync(0xffffffffu, key, (int)(src[j >> 2] >> (8 * (j & 3))));
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < CMAX; ++j) cnt += other[j] < key ? 1 : 0;
    if (cnt < k && (int32_t)key >= 0) {
      Le32 += 32;
      sel[base + cnt] = (uint8_t)(add & 31u);
    }
  }
}

// Chain over one tile's list, lane = candidate, loads in shared memory.
template <int CMAX>
__device__ __forceinline__ void k2_chain_cands(int32_t* L, const uint32_t* list, int n_dec, int k,
                                               int LW, int EW, uint8_t* sel, int lane) {
  const bool has = lane < LW;
  uint32_t w_n = has ? list[lane] : 0x8000u, base_n = list[LW + 4];
#pragma unroll 1
  for (int i = 0; i < n_dec; ++i) {
    const uint32_t w = w_n, base = base_n;
    const uint32_t* nx = list + (i + 1) * EW;   // the list has one spare entry
    if (has) w_n = nx[lane];
    base_n = nx[LW + 4];
    const bool cand = (w & 0x8000u) == 0;
    const int id = (int)(w >> 16);
    const int32_t Lraw = L[id];
    const uint32_t key = cand ? ((uint32_t)Lraw << 5) + (w & 0x7fffu) : 0xffffffffu;
    uint32_t other[CMAX];
#pragma unroll
    for (int j = 0; j < CMAX; ++j) other[j] = __shfl_sync(0xffffffffu, key, j);
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < CMAX; ++j) cnt += other[j] < key ? 1 : 0;
    if (cand && cnt < k) {
      L[id] = Lraw + 1;
      sel[base + cnt] = (uint8_t)lane;
    }
    __syncwarp();
  }
}

// Fallback for candidate sets or k wider than a warp, or loads of 2^25 and more: one warp
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

// Selection role of one thread block (kK2Threads threads) for one layer, tokens
// [A.tok_begin, A.tok_end).  smem: k2_smem_bytes().  When ready != nullptr the records are
// produced concurrently by router blocks of the same launch, which publish one flag per
// router_rows tokens; a wait that runs out raises LASER_DEV_TIMEOUT and ends the role.
__device__ __forceinline__ void k2_block(const RouteArgs& A, int layer, unsigned char* k2_smem,
                                         const int* ready, int router_rows) {
  __shared__ int s_tile_ok[2];
  int my_abort = 0;   // set by the thread whose wait ran out; made uniform at the barriers
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
      bool ok = true;
      for (int t0 = 0; t0 < ntot && ok; t0 += router_rows) {
        const int n = min(router_rows, ntot - t0);
        if (ready) {
          int good = 1;
          if (lane == 0) good = k2_wait_ready(ready, router_rows, tb + t0, tb + t0 + n - 1) ? 1 : 0;
          ok = __shfl_sync(0xffffffffu, good, 0) != 0;
          if (!ok) break;
        }
        k2_chain_wide(L, keys, g_cs + t0, g_ids + (size_t)t0 * c, g_sel + (size_t)t0 * k, n, k, c,
                      lane);
      }
      if (!ok && lane == 0 && A.status) atomicOr(A.status, 2);
      for (int e = lane; e < E; e += 32) g_loads[e] = L[e];
    }
    return;
  }
  const bool small_e = E <= 32 && c <= 16;
  const int Ew = E > 32 ? E : 32;
  const int LW = k2_lane_words(E, c), EW = k2_entry_words(E, c);
  const int n_tiles = (ntot + kK2Tile - 1) / kK2Tile;

  // Tile preparation by warps [first_warp, first_warp + n_warps); bar_id names their barrier.
  auto prep_tile = [&](int tile, int first_warp, int n_warps, int bar_id) {
    const K2Buffers b = k2_carve(buf0 + (size_t)(tile & 1) * buf_bytes, E, c);
    const int t0 = tile * kK2Tile;
    int ntok = min(kK2Tile, ntot - t0);
    const int w = warp - first_warp;
    if (ready) {
      if (w == 0 && lane == 0) {
        const bool ok = k2_wait_ready(ready, router_rows, tb + t0, tb + t0 + ntok - 1);
        s_tile_ok[tile & 1] = ok ? 1 : 0;
        if (!ok) { my_abort = 1; if (A.status) atomicOr(A.status, 2); }
      }
      named_barrier(bar_id, n_warps * 32);
      if (!s_tile_ok[tile & 1]) ntok = 0;   // an unpublished tile is treated as empty
    }
    const int n_groups = (ntok + 31) >> 5;
    for (int g = w; g < n_groups; g += n_warps)
      k2_stage_group(b, g, ntok, g_ids + (size_t)t0 * c, g_cs + t0, c, lane);
    cp_async_wait_all();
    __syncwarp();
    for (int g = w; g < n_groups; g += n_warps)
      k2_count_group(b, g, ntok, E, Ew, k, c, small_e, lane);
    for (int g = n_groups + w; g < kK2Groups; g += n_warps)
      if (lane == 0) b.dcount[g] = 0;
    named_barrier(bar_id, n_warps * 32);
    // exclusive prefix of the fixed increments over the groups, and the tile totals
    for (int e = w * 32 + lane; e < E; e += n_warps * 32) {
      int32_t run = 0;
      for (int g = 0; g < n_groups; ++g) {
        const int32_t v = small_e ? __popc(b.gB[g * 32 + e]) : b.gtot[g * Ew + e];
        b.gtot[g * Ew + e] = run;
        run += v;
      }
      b.ttot[e] = run;
    }
    named_barrier(bar_id, n_warps * 32);
    for (int g = w; g < n_groups; g += n_warps) {
      if (k <= 8) k2_list_group<8>(b, g, ntok, E, Ew, k, c, small_e, LW, EW, lane);
      else k2_list_group<0>(b, g, ntok, E, Ew, k, c, small_e, LW, EW, lane);
    }
  };

  if (n_tiles > 0) prep_tile(0, 0, kK2Warps, 1);
  bool stop = __syncthreads_or(my_abort) != 0;
  uint32_t Le32 = (warp == 0 && lane < E) ? (uint32_t)L[lane] << 5 : 0;
  for (int tile = 0; tile < n_tiles && !stop; ++tile) {
    if (warp > 0) {
      if (tile + 1 < n_tiles) prep_tile(tile + 1, 1, kK2Warps - 1, 2);
    } else {
      const K2Buffers b = k2_carve(buf0 + (size_t)(tile & 1) * buf_bytes, E, c);
      uint8_t* sel = g_sel + (size_t)tile * kK2Tile * k;
      int n_dec = lane < kK2Groups ? b.dcount[lane] : 0;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) n_dec += __shfl_xor_sync(0xffffffffu, n_dec, s);
      if (small_e) {
        if (c <= 4) k2_chain_experts<4>(Le32, b.list, n_dec, k, LW, EW, sel, lane);
        else if (c <= 8) k2_chain_experts<8>(Le32, b.list, n_dec, k, LW, EW, sel, lane);
        else k2_chain_experts<16>(Le32, b.list, n_dec, k, LW, EW, sel, lane);
        if (lane < E) Le32 += (uint32_t)b.ttot[lane] << 5;
      } else {
        if (c <= 8) k2_chain_cands<8>(L, b.list, n_dec, k, LW, EW, sel, lane);
        else if (c <= 16) k2_chain_cands<16>(L, b.list, n_dec, k, LW, EW, sel, lane);
        else k2_chain_cands<32>(L, b.list, n_dec, k, LW, EW, sel, lane);
        for (int e = lane; e < E; e += 32) L[e] += b.ttot[e];
        __syncwarp();
      }
    }
    stop = __syncthreads_or(my_abort) != 0;
  }
  if (small_e) {
    if (warp == 0 && lane < E) g_loads[lane] = (int32_t)(Le32 >> 5);
  } else {
    for (int e = tid; e < E; e += kK2Threads) g_loads[e] = L[e];
  }
}

}  // namespace laser
