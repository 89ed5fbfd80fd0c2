// K2: the ordered, load-aware selection (Algorithm 1, StableSortByLoad + first k) and the
// per-token load update.  Tokens of one layer form one dependency chain; layers are
// independent thread blocks.
//
// The rule is sequential: token t sees the loads left by tokens 0..t-1.  The block handles a
// batch of 256 consecutive tokens at a time, thread = token, by iterating to the fixed point of
//     choice_i = k smallest (load at batch start + #{j < i : e in choice_j}, score rank)
// starting from "every token takes its k best".  A sweep recomputes the per-expert prefix
// counts from the current choices and lets every token with a load-dependent choice (c* > k)
// choose again.  After sweep n the first n tokens of the batch hold their sequential choice
// (token i only depends on tokens j < i), so a sweep that changes nothing has reached exactly
// the sequential result; it comes after at most 257 sweeps and typically after two or three,
// because the increments inside a batch rarely reorder the candidates' loads (when all loads
// are tied, as under load-only routing, a batch needs a few dozen).  Tokens on the top-k
// branch or with c* == k never change their choice; they only contribute increments.
//   E <= 32   a choice is a bit mask over experts; per warp one ballot per expert gives the
//             tokens that chose it (kept by lane = expert), warp totals go through shared
//             memory, and a candidate's prefix count comes back by shuffle.
//   E  > 32   one 32-bit "who chose me" mask per (warp, expert) in shared memory, maintained
//             with atomics by the tokens that change, and their exclusive prefix over warps.
//             Under the rule's own order the fixed point is not iterated: the tokens without
//             a decision are counted in parallel, the load every candidate of every decision
//             token would see without the batch's decisions is worked out in parallel, and
//             warp 0 takes the decision tokens one after the other (lane = candidate), adding
//             the decisions made so far.  The sweeps serve the relaxed granularities.
// The candidates' keys (load << 5 | score rank) are sorted by a compile-time bitonic network
// over CMAX registers; the first k give the choice in the order the method lists it.
// Per group of 32 tokens the block stores how many assignments of this call preceded the
// group per expert; the dispatch kernel turns those into stable positions.  At the end the
// block writes the loads, this call's offsets (exclusive scan of the counts) and the
// device-bin sums.
#pragma once
#include "laser_common.cuh"
#include "k2_chain.cuh"
#include "k3_dispatch.cuh"

namespace laser {

constexpr int kK2Threads = 256;
constexpr int kK2Warps = kK2Threads / 32;
constexpr int kK2Batch = kK2Threads;     // tokens per batch, thread = token
constexpr int kK2FastMaxLoad = 1 << 25;  // 32-bit keys (load << 5 | rank) stay below 2^31
constexpr int kK2MaxSweeps = kK2Batch + 2;
constexpr long long kK2WaitCycles = 4000000000LL;  // default limit of a wait: ~2 s

__host__ __device__ inline bool k2_fast_shape(int k, int c) { return c <= 32 && k <= 32; }
__host__ __device__ inline size_t k2_batch_bytes(int c) {
  return align256((size_t)kK2Batch * sizeof(uint16_t)) + align256((size_t)kK2Batch * c);
}

// Shared memory of the selection role:
//   int32 L[E] | int32 Lin[E] | int32 Lvis[E] | uint64 keys[c] | int32 wtot[8][max(E,32)] |
//   then either the batch fixed point's part
//     uint32 mask[8][E] | int32 excl[8][E] | uint8 chosen[256][32] (all three E > 32 only) |
//     2 batch buffers (c*, candidate ids)
//   or (E > 32, the rule's own update order) the pipeline's part, k2_chain_smem_bytes()
__host__ __device__ inline size_t k2_smem_bytes(int E, int c, int k) {
  const size_t Ew = E > 32 ? E : 32;
  const size_t b = 3 * align256(sizeof(int32_t) * E) + align256(sizeof(unsigned long long) * c) +
                   align256(sizeof(int32_t) * kK2Warps * Ew);
  if (!k2_fast_shape(k, c)) return b;
  size_t sweeps = 2 * k2_batch_bytes(c);
  if (E <= 32) return b + sweeps;
  sweeps += 2 * align256(sizeof(int32_t) * kK2Warps * E) + (size_t)kK2Batch * 32;
  const size_t chain = k2_chain_smem_bytes(E, c);
  return b + (sweeps > chain ? sweeps : chain);
}

// Calls of at most this many 32-token groups have their dispatch done by the selection block
// itself (one launch less); its scratch lies behind L, Lin and Lvis in the selection's memory.
constexpr int kFusedDispatchGroups = 16;
__host__ __device__ inline size_t k2_fused_dispatch_bytes(int E, int k) {
  return 3 * align256(sizeof(int32_t) * E) + (size_t)kK2Warps * k3_warp_smem_bytes(E, k);
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_all;" ::: "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Called by one full warp: waits until the router blocks that produce tokens
// [t_first, t_last] of this layer have published their records (the lanes share the flags).
// Bounded: gives up after `limit` cycles and returns false; also false as soon as one of the
// tiles reports that it gave up itself (flag < 0).  block = false only tests once.
__device__ __forceinline__ bool k2_wait_ready(const int* ready, int router_rows, int t_first,
                                              int t_last, long long limit, bool block) {
  const int lane = threadIdx.x & 31;
  const int rt0 = t_first / router_rows, rt1 = t_last / router_rows;
  const long long start = clock64();
  for (int base = rt0; base <= rt1; base += 32) {
    const int rt = base + lane;
    while (true) {
      const int v = rt > rt1 ? 1 : ld_acquire(ready + rt);
      if (__any_sync(0xffffffffu, v < 0)) return false;
      if (__all_sync(0xffffffffu, v != 0)) break;
      if (!block || clock64() - start > limit) return false;
      __nanosleep(100);
    }
  }
  return true;
}

// Ascending bitonic sort of N (power of two) registers; every index is a compile-time value.
template <int N>
__device__ __forceinline__ void sort_keys(uint32_t (&a)[N]) {
#pragma unroll
  for (int size = 2; size <= N; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const int j = i ^ stride;
        if (j > i) {
          const uint32_t lo = min(a[i], a[j]), hi = max(a[i], a[j]);
          const bool up = (i & size) == 0;
          a[i] = up ? lo : hi;
          a[j] = up ? hi : lo;
        }
      }
    }
  }
}

struct K2Smem {
  int32_t* L;        // [E] loads at the start of the current batch
  int32_t* Lin;      // [E] loads on entry
  int32_t* Lvis;     // [E] relaxed variant: loads at the start of the chunk that reaches
                     //     into the current batch from an earlier one
  unsigned long long* keys;  // [c] slow scan only
  int32_t* wtot;     // [8][max(E,32)] per warp and expert: tokens of the warp that chose it
  uint32_t* mask;    // [8][E]  E > 32: bit i = token i of the warp chose this expert
  int32_t* excl;     // [8][E]  E > 32: exclusive prefix of the mask popcounts over warps
  uint8_t* chosen;   // [256][32] E > 32: current choice of every token, key order
};

// One batch of up to 256 tokens, thread = token, run by the whole block.
// cs_s / ids_s: the batch's staged c* and ranked ids.  On return sm.L has advanced past the
// batch, the decision tokens' chosen ranks are in sel ([256][k], batch-relative) and
// g_base ([8][E], batch-relative groups) holds, per group of 32 tokens and expert, the
// assignments of this call made before the group.
template <int CMAX, bool SMALL>
__device__ __forceinline__ void k2_batch(const K2Smem& sm, const uint16_t* cs_s,
                                         const uint8_t* ids_s, int n_here, int E, int k, int c,
                                         uint8_t* sel, int32_t* g_base, int G, int t0) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Ew = E > 32 ? E : 32;
  // Relaxed variant (G != 1; G is 0 or a multiple of 32, so a warp's 32 tokens share a chunk):
  // a token sees the loads at the start of its chunk.  If the chunk began in an earlier batch
  // those are sm.Lvis and nothing of this batch; otherwise sm.L plus the choices of the warps
  // before the chunk's first warp wc.
  const bool strict = G == 1;
  const int c0 = G == 0 ? 0 : ((t0 + warp * 32) / (G > 0 ? G : 1)) * G;   // chunk start (token)
  const bool outside = !strict && c0 < t0;
  const int wc = (strict || outside) ? 0 : (c0 - t0) / 32;
  const bool valid = tid < n_here;
  const int cs = valid ? cs_s[tid] : 0;
  const bool dec = cs > k;
  const uint8_t* my = ids_s + tid * c;
  const unsigned below = (1u << lane) - 1;
  const int n_dec = __syncthreads_count(dec);   // also: sm.L of the previous batch is final
  const bool any_dec = n_dec != 0;
  int32_t* wt = sm.wtot + warp * Ew;

  if (SMALL) {
    uint32_t m = 0;    // current choice as a bit mask over experts; the k best to start with
    if (valid)
      for (int j = 0; j < k; ++j) m |= 1u << my[j];
    uint32_t Bm = 0;   // lane e: which tokens of this warp currently choose expert e
    int32_t excl = 0;  // lane e: tokens of earlier warps that currently choose expert e
    int cid[CMAX];
    uint32_t Lc[CMAX], key[CMAX];
    if (any_dec) {
#pragma unroll
      for (int r = 0; r < CMAX; ++r) {
        cid[r] = (dec && r < cs) ? my[r] : 0;
        Lc[r] = (uint32_t)(outside ? sm.Lvis[cid[r]] : sm.L[cid[r]]);
      }
    }
    for (int sweep = 0; sweep < kK2MaxSweeps; ++sweep) {
      for (int e = 0; e < E; ++e) {
        const uint32_t B = __ballot_sync(0xffffffffu, (m >> e) & 1u);
        if (lane == e) Bm = B;
      }
      wt[lane] = __popc(Bm);
      __syncthreads();
      excl = 0;
      int32_t exv = 0;   // relaxed: choices of the warps before the chunk's first warp
      for (int w = 0; w < warp; ++w) {
        const int32_t v = sm.wtot[w * Ew + lane];
        excl += v;
        if (w < wc) exv += v;
      }
      if (!any_dec) break;
      uint32_t m_new = m;
#pragma unroll
      for (int r = 0; r < CMAX; ++r) {
        const uint32_t Br = __shfl_sync(0xffffffffu, Bm, cid[r]);
        const uint32_t ex = (uint32_t)__shfl_sync(0xffffffffu, strict ? excl : exv, cid[r]);
        const uint32_t seen = Lc[r] + ex + (strict ? (uint32_t)__popc(Br & below) : 0u);
        key[r] = (dec && r < cs) ? ((seen << 5) | (uint32_t)r) : 0xffffffffu;
      }
      if (dec) {
        sort_keys<CMAX>(key);
        m_new = 0;
#pragma unroll
        for (int j = 0; j < CMAX; ++j)
          if (j < k) m_new |= 1u << my[key[j] & 31u];
      }
      const bool changed = m_new != m;
      m = m_new;
      if (!__syncthreads_or(changed)) break;   // Bm, excl and wtot describe the final choices
    }
    if (dec) {
#pragma unroll
      for (int j = 0; j < CMAX; ++j)
        if (j < k) sel[tid * k + j] = (uint8_t)(key[j] & 31u);
    }
    if (lane < E && warp * 32 < n_here)
      g_base[warp * E + lane] = sm.L[lane] - sm.Lin[lane] + excl;
    __syncthreads();   // every thread has read sm.L, sm.Lvis and wtot
    if (warp == 0 && lane < E) {
      // relaxed: the chunk that holds the next batch's first token, if it began in this batch
      const int t_next = t0 + kK2Batch;
      const int c_next = G == 0 ? 0 : (t_next / (G > 0 ? G : 1)) * G;
      const int wl = (c_next - t0) / 32;
      int32_t tot = 0, upto = 0;
      for (int w = 0; w < kK2Warps; ++w) {
        const int32_t v = sm.wtot[w * Ew + lane];
        tot += v;
        if (w < wl) upto += v;
      }
      if (!strict && c_next >= t0) sm.Lvis[lane] = sm.L[lane] + (c_next < t_next ? upto : tot);
      sm.L[lane] += tot;
    }
    return;   // the next batch starts with a barrier
  }

  // E > 32: per (warp, expert) masks in shared memory (all zero between batches)
  uint32_t* mk = sm.mask + warp * E;
  uint8_t* ch = sm.chosen + tid * 32;

  if (valid)   // every token takes its k best to start with
    for (int j = 0; j < k; ++j) {
      ch[j] = my[j];
      atomicOr(&mk[my[j]], 1u << lane);
    }
  int cid[CMAX];
  uint32_t Lc[CMAX], key[CMAX];
  if (any_dec) {
#pragma unroll
    for (int r = 0; r < CMAX; ++r) {
      cid[r] = (dec && r < cs) ? my[r] : 0;
      Lc[r] = (uint32_t)(outside ? sm.Lvis[cid[r]] : sm.L[cid[r]]);
    }
  }
  for (int sweep = 0; sweep < kK2MaxSweeps; ++sweep) {
    __syncthreads();   // masks of this sweep are complete
    for (int e = tid; e < E; e += kK2Threads) {
      int32_t run = 0;
#pragma unroll
      for (int w = 0; w < kK2Warps; ++w) {
        sm.excl[w * E + e] = run;
        run += __popc(sm.mask[w * E + e]);
      }
      sm.wtot[e] = run;   // batch total per expert
    }
    __syncthreads();
    if (!any_dec) break;
    bool changed = false;
    if (dec) {
#pragma unroll
      for (int r = 0; r < CMAX; ++r)
        key[r] = r < cs ? (((Lc[r] +
                             (strict ? (uint32_t)sm.excl[warp * E + cid[r]] +
                                           (uint32_t)__popc(mk[cid[r]] & below)
                                     : (outside ? 0u : (uint32_t)sm.excl[wc * E + cid[r]])))
                            << 5) | (uint32_t)r)
                        : 0xffffffffu;
      sort_keys<CMAX>(key);
#pragma unroll
      for (int j = 0; j < CMAX; ++j)
        if (j < k) changed |= (my[key[j] & 31u] != ch[j]);
    }
    if (!__syncthreads_or(changed)) break;   // also: every thread has read this sweep's masks
    if (changed)
      for (int j = 0; j < k; ++j) atomicAnd(&mk[ch[j]], ~(1u << lane));
    __syncwarp();
    if (changed) {
#pragma unroll
      for (int j = 0; j < CMAX; ++j)
        if (j < k) {
          const uint8_t e = my[key[j] & 31u];
          ch[j] = e;
          atomicOr(&mk[e], 1u << lane);
        }
    }
  }
  if (dec) {
#pragma unroll
    for (int j = 0; j < CMAX; ++j)
      if (j < k) sel[tid * k + j] = (uint8_t)(key[j] & 31u);
  }
  for (int i = tid; i < kK2Warps * E; i += kK2Threads) {
    const int e = i % E;
    if ((i / E) * 32 < n_here) g_base[i] = sm.L[e] - sm.Lin[e] + sm.excl[i];
  }
  __syncthreads();   // every thread has read the masks, excl, sm.L and sm.Lvis of this batch
  {
    const int t_next = t0 + kK2Batch;
    const int c_next = G == 0 ? 0 : (t_next / (G > 0 ? G : 1)) * G;
    const int wl = (c_next - t0) / 32;
    for (int e = tid; e < E; e += kK2Threads) {
      if (!strict && c_next >= t0)
        sm.Lvis[e] = sm.L[e] + (c_next < t_next ? sm.excl[wl * E + e] : sm.wtot[e]);
      sm.L[e] += sm.wtot[e];
    }
  }
  for (int i = tid; i < kK2Warps * E; i += kK2Threads) sm.mask[i] = 0;
}

// Slow scan for candidate sets or k wider than a warp, or loads of 2^25 and more: one warp
// walks every token of one group; 64-bit keys (load, score rank) go through shared memory.
__device__ __forceinline__ void k2_wide_group(int32_t* L, const int32_t* Lsee,
                                              unsigned long long* keys,
                                              const uint16_t* g_cs, const uint8_t* g_ids,
                                              uint8_t* g_sel, int ntok, int k, int c, int lane) {
  for (long long t = 0; t < ntok; ++t) {
    const int cs = g_cs[t];
    const uint8_t* ids = g_ids + t * c;
    if (cs <= k) {
      for (int j = lane; j < k; j += 32) L[ids[j]] += 1;
    } else {
      for (int j = lane; j < cs; j += 32)
        keys[j] = (((unsigned long long)(uint32_t)Lsee[ids[j]]) << 8) | (unsigned)j;
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

// Selection role of one thread block (kK2Threads threads) for one layer (absolute index),
// templated on the sorting width CMAX >= c (32 also serves the slow scan) and on SMALL
// (E <= 32).
// smem: k2_smem_bytes().  When ready != nullptr the records are produced concurrently by
// router blocks of the same launch, which publish one flag per router_rows tokens; a wait that
// runs out raises LASER_DEV_TIMEOUT and ends the role.
template <int CMAX, bool SMALL>
__device__ __forceinline__ void k2_block(const RouteArgs& A, int layer, unsigned char* k2_smem,
                                         const int* ready, int router_rows) {
  __shared__ int s_flag;      // outcome of a blocking wait for the router
  __shared__ int s_gave_up;   // a wait ran out: the layer is aborted
  __shared__ int s_next[2];   // [b & 1]: batch b + 1 was prefetched during batch b
  const int E = A.E, k = A.k, c = A.c, T = A.T;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Ew = E > 32 ? E : 32;

  K2Smem sm;
  unsigned char* p = k2_smem;
  sm.L = reinterpret_cast<int32_t*>(p);       p += align256(sizeof(int32_t) * E);
  sm.Lin = reinterpret_cast<int32_t*>(p);     p += align256(sizeof(int32_t) * E);
  sm.Lvis = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * E);
  sm.keys = reinterpret_cast<unsigned long long*>(p);  p += align256(sizeof(unsigned long long) * c);
  sm.wtot = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * kK2Warps * Ew);
  sm.mask = nullptr; sm.excl = nullptr; sm.chosen = nullptr;
  unsigned char* chain_smem = p;   // E > 32 under the rule's own order: the pipeline's part
  const bool chain = E > 32 && A.G == 1 && k2_fast_shape(k, c);
  if (E > 32 && k2_fast_shape(k, c) && !chain) {
    sm.mask = reinterpret_cast<uint32_t*>(p);  p += align256(sizeof(int32_t) * kK2Warps * E);
    sm.excl = reinterpret_cast<int32_t*>(p);   p += align256(sizeof(int32_t) * kK2Warps * E);
    sm.chosen = p;                              p += (size_t)kK2Batch * 32;
  }
  unsigned char* bufs = p;
  const size_t buf_bytes = k2_batch_bytes(c);

  unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const uint16_t* g_cs = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar);
  const uint8_t* g_ids = ws + A.lay.cand_ids;
  uint8_t* g_sel = ws + A.lay.sel_rank;
  int32_t* g_base = reinterpret_cast<int32_t*>(ws + A.lay.grp_base);
  int32_t* g_loads = A.loads + (size_t)layer * E;
  const int n_groups = A.lay.n_groups;

  if (sm.mask)
    for (int i = tid; i < kK2Warps * E; i += kK2Threads) sm.mask[i] = 0;
  if (tid == 0) s_gave_up = 0;
  // A wait that runs out (or a router tile that gave up) aborts the layer: the status bit is
  // raised and the layer's abort word set, after which neither this block nor the dispatch
  // reads the layer's scratch records again (they may be unwritten).
  // (the layer's control words live behind its ready flags; without flags -- the records are
  // all there when the block starts -- nothing cleared them, so this block does)
  int* ctrl = reinterpret_cast<int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready);
  int* abort_word = ctrl + abort_word_index(T);
  if (!ready && tid == 0) *abort_word = 0;
  auto give_up = [&]() {
    if (A.status) atomicOr(A.status, 2);
    st_release(abort_word, 1);
    s_gave_up = 1;
  };
  int too_big = 0;
  for (int e = tid; e < E; e += kK2Threads) {
    const int32_t v = A.fresh ? 0 : g_loads[e];
    sm.L[e] = v;
    sm.Lin[e] = v;
    sm.Lvis[e] = v;
    // a counter within T of 2^31-1 could wrap during the call: raise the status bit
    if (v < 0 || v > 0x7fffffff - T) { if (A.status) atomicOr(A.status, 1); }
    if (v < 0 || v > kK2FastMaxLoad - T) too_big = 1;
  }
  const bool wide = __syncthreads_or(too_big) || !k2_fast_shape(k, c);
  // how the decision tokens' choices are left for the dispatch: rank masks (1) or rank lists (0)
  if (tid == 0) ctrl[mode_word_index(T)] = (!wide && !SMALL && chain) ? 1 : 0;

  if (wide) {
    if (warp == 0) {
      bool ok = true;
      for (int g = 0; g < n_groups && ok; ++g) {
        const int t0 = g * 32, n = min(32, T - t0);
        // the whole group must be there: a router tile may be shorter than a group (16 tokens
        // with the split-K router) or span several groups
        if (ready && (router_rows < 32 || (t0 % router_rows) == 0)) {
          ok = k2_wait_ready(ready, router_rows, t0, min(T, t0 + max(32, router_rows)) - 1,
                             A.wait_cycles);
          if (!ok) break;
        }
        for (int e = lane; e < E; e += 32) g_base[(size_t)g * E + e] = sm.L[e] - sm.Lin[e];
        if (A.G != 1 && (A.G == 0 ? t0 == 0 : t0 % A.G == 0)) {   // relaxed: a chunk begins
          for (int e = lane; e < E; e += 32) sm.Lvis[e] = sm.L[e];
          __syncwarp();
        }
        k2_wide_group(sm.L, A.G == 1 ? sm.L : sm.Lvis, sm.keys, g_cs + t0, g_ids + (size_t)t0 * c,
                      g_sel + (size_t)t0 * k, n, k, c, lane);
      }
      if (!ok && lane == 0) give_up();
    }
  } else if (!SMALL && chain) {
    k2_chain_layer<CMAX>(A, layer, chain_smem, sm.L, sm.Lin, &s_gave_up, ready, router_rows,
                         give_up);
  } else {
    const int n_batches = (T + kK2Batch - 1) / kK2Batch;
    // copies the c* and candidate ids of batch b into buffer b & 1 (cp.async, not waited for)
    auto stage = [&](int b) {
      const int t0 = b * kK2Batch, nt = min(kK2Batch, T - t0);
      unsigned char* dst = bufs + (size_t)(b & 1) * buf_bytes;
      const unsigned char* src_cs = reinterpret_cast<const unsigned char*>(g_cs + t0);
      const unsigned char* src_ids = g_ids + (size_t)t0 * c;
      unsigned char* dst_ids = dst + align256((size_t)kK2Batch * sizeof(uint16_t));
      for (int i = tid; i < (nt * 2 + 15) / 16; i += kK2Threads)
        cp_async16(dst + 16 * i, src_cs + 16 * i);
      for (int i = tid; i < (nt * c + 15) / 16; i += kK2Threads)
        cp_async16(dst_ids + 16 * i, src_ids + 16 * i);
    };
    // the same copy issued by the last warp alone, for the batch after the current one
    auto stage_by_warp = [&](int b) {
      const int t0 = b * kK2Batch, nt = min(kK2Batch, T - t0);
      unsigned char* dst = bufs + (size_t)(b & 1) * buf_bytes;
      const unsigned char* src_cs = reinterpret_cast<const unsigned char*>(g_cs + t0);
      const unsigned char* src_ids = g_ids + (size_t)t0 * c;
      unsigned char* dst_ids = dst + align256((size_t)kK2Batch * sizeof(uint16_t));
      for (int i = lane; i < (nt * 2 + 15) / 16; i += 32) cp_async16(dst + 16 * i, src_cs + 16 * i);
      for (int i = lane; i < (nt * c + 15) / 16; i += 32)
        cp_async16(dst_ids + 16 * i, src_ids + 16 * i);
    };
    // The last warp looks ahead for the router's flags: those of batch b + 1 are loaded while
    // batch b - 1 is processed and first used a whole batch later, so the latency of the loads
    // is not on the path of any batch.  (A flag seen unset is simply looked at again by the
    // blocking wait.)
    auto load_flags = [&](int b1) -> int {
      int f = 1;
      if (ready && b1 < n_batches) {
        const int t1 = b1 * kK2Batch, n1 = min(kK2Batch, T - t1);
        const int rt = t1 / router_rows + lane;      // at most 16 flags per batch
        if (rt <= (t1 + n1 - 1) / router_rows) f = ld_acquire(ready + rt);
      }
      return f;
    };
    const bool looker = warp == kK2Warps - 1;
    int flag_next = looker ? load_flags(1) : 1;   // flags of batch b + 1
    bool staged = false;   // batch b is already on its way into its buffer
    for (int b = 0; b < n_batches; ++b) {
      const int t0 = b * kK2Batch, nt = min(kK2Batch, T - t0);
      if (!staged) {
        if (ready) {
          if (warp == 0) {
            const bool good = k2_wait_ready(ready, router_rows, t0, t0 + nt - 1, A.wait_cycles);
            if (lane == 0) s_flag = good ? 1 : 0;
          }
          __syncthreads();
          if (!s_flag) {
            if (tid == 0) give_up();
            break;
          }
        }
        stage(b);
      }
      const bool look = looker && b + 1 < n_batches;
      const int flag_after = looker ? load_flags(b + 2) : 1;   // used in the next iteration
      cp_async_wait_all();
      __syncthreads();   // batch b is in shared memory
      if (look) {
        const bool okn = __all_sync(0xffffffffu, flag_next > 0);
        if (okn) stage_by_warp(b + 1);
        if (lane == 0) s_next[b & 1] = okn ? 1 : 0;
      }
      flag_next = flag_after;
      const unsigned char* buf = bufs + (size_t)(b & 1) * buf_bytes;
      k2_batch<CMAX, SMALL>(sm, reinterpret_cast<const uint16_t*>(buf),
                                   buf + align256((size_t)kK2Batch * sizeof(uint16_t)), nt, E, k,
                                   c, g_sel + (size_t)t0 * k, g_base + (size_t)(t0 / 32) * E, A.G,
                                   t0);
      // written before the barriers inside k2_batch; rewritten two batches later
      staged = b + 1 < n_batches && s_next[b & 1] != 0;
    }
  }
  __syncthreads();

  // loads out, offsets = exclusive scan of this call's counts, device-bin sums
  __shared__ int32_t s_cnt[kMaxExperts];
  __shared__ int32_t s_warp_tot[kK2Warps];
  int32_t cnt = 0;
  if (tid < E) {
    cnt = sm.L[tid] - sm.Lin[tid];
    s_cnt[tid] = cnt;
    g_loads[tid] = sm.L[tid];
  }
  int32_t incl = cnt;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const int32_t up = __shfl_up_sync(0xffffffffu, incl, s);
    if (lane >= s) incl += up;
  }
  if (lane == 31) s_warp_tot[warp] = incl;
  __syncthreads();
  int32_t before = 0;
  for (int w = 0; w < warp; ++w) before += s_warp_tot[w];
  int32_t* offsets = A.offsets + (size_t)layer * (E + 1);
  __shared__ int32_t s_off[kMaxExperts + 1];
  if (tid < E) {
    offsets[tid] = s_off[tid] = before + incl - cnt;
    if (tid == E - 1) offsets[E] = s_off[E] = before + incl;
  }
  if (A.bin_loads) {
    const int B = A.n_bins;
    const int per = (E + B - 1) / B;
    int32_t* bl = A.bin_loads + (size_t)layer * B;
    for (int b = tid; b < B; b += kK2Threads) {
      int32_t s = 0;
      for (int e = 0; e < E; ++e) {
        const int be = A.e2b ? A.e2b[e] : e / per;
        if (be == b) s += s_cnt[e];
      }
      bl[b] = (A.fresh ? 0 : bl[b]) + s;
    }
  }
  if (A.fuse_dispatch && !s_gave_up) {   // (s_gave_up was written before the barriers above)
    // few groups: the dispatch of this layer here, instead of one more launch.  The barrier makes
    // the offsets and this block's chosen ranks and group base counts visible to all its warps;
    // the routers' records were acquired with their flags.
    __syncthreads();
    unsigned char* scratch = k2_smem + 3 * align256(sizeof(int32_t) * E);
    for (int g = warp; g < n_groups; g += kK2Warps)
      k3_group(A, layer, g, sm.Lin, s_off, scratch + (size_t)warp * k3_warp_smem_bytes(E, k));
  }
}

}  // namespace laser
