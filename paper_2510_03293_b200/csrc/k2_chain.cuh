// K2 for E > 32 under the method's own load update (after every token): the ordered selection
// of one layer as a pipeline inside one thread block.
//
// What a token with a load-dependent choice (c* > k, a "decision token") has to know is, for
// each of its candidates e, the load e has when the token's turn comes:
//     L_in[e] + (assignments to e by earlier tokens that have no decision to take)
//             + (assignments to e by earlier decision tokens).
// Only the last term depends on the loads.  The router blocks publish, per group of 32 tokens
// and expert, the bit mask of the group's tokens without a decision that go to that expert
// ("fixed" tokens: top-k branch or c* == k; they take their k best whatever the loads are).
//
// Helper warps 1..7 each prepare every seventh group, ahead of the chain:
//   - the group's masks and c* / candidate records come in from global memory (requested one
//     round ahead when the router has already published them),
//   - the running per-expert count of fixed assignments is handed from group to group in order
//     (the one serial step of the helpers: E additions),
//   - every decision token of the group becomes one entry of CMAX 8-byte words, lane =
//     candidate: the first two terms above | the candidate's expert | the lane of the group's
//     previous entry that holds the same expert (if any) | the token.
// Warp 0, the chain, walks the groups in order and their entries one after the other:
//     key = (first two terms + decisions so far for the expert) << 5 | score rank,
//     rank of the key among the entry's keys by all-pairs comparison (shuffles),
//     the k smallest are the choice; their experts' decision counters go up by one.
// The decision counters live in shared memory.  To keep their read off the critical path the
// counter of the next entry's candidates is read before the current entry's increments and
// corrected by the current choice through the prepared cross-reference (one ballot).  The
// choice of an entry is a bit mask over its candidates; the helper that owns the slot copies
// the masks to global memory when it next visits the slot.  At every group boundary the chain
// writes the group's base counts (fixed prefix + decisions so far) that the dispatch turns
// into positions.  All hand-overs are sequence numbers in shared memory; the waits for the
// router are bounded, and a wait that runs out ends every role.
#pragma once
#include "laser_common.cuh"

namespace laser {

constexpr int kChainSlots = 7;   // helper warps = groups in preparation

// (defined with the rest of the selection role) waits, bounded, for the router's flags of tokens
// [t_first, t_last]; called by a full warp
__device__ __forceinline__ bool k2_wait_ready(const int* ready, int router_rows, int t_first,
                                              int t_last, long long limit, bool block = true);

__host__ __device__ inline int chain_cmax(int c) { return c <= 4 ? 4 : (c <= 8 ? 8 : (c <= 16 ? 16 : 32)); }
// one slot: fb[E] int32 | db[E] int32 | fm[E] uint32 | ent[32][CMAX] u64 | ids[32][CMAX] u8 |
// out[32] u32 | n, seq, dl[32]
__host__ __device__ inline size_t k2_chain_slot_bytes(int E, int cmax) {
  return 3 * align256(sizeof(int32_t) * E) + (size_t)32 * cmax * 8 + (size_t)32 * cmax + 128 + 128;
}
// dcnt[E] | fcum[E] | counters | slots
__host__ __device__ inline size_t k2_chain_smem_bytes(int E, int c) {
  return 2 * align256(sizeof(int32_t) * E) + 256 + kChainSlots * k2_chain_slot_bytes(E, chain_cmax(c));
}

__device__ __forceinline__ int ld_volatile_shared(const int* p) {
  return *reinterpret_cast<const volatile int*>(p);
}
__device__ __forceinline__ void st_volatile_shared(int* p, int v) {
  *reinterpret_cast<volatile int*>(p) = v;
}
// shared-memory accesses by 32-bit shared address (the chain's inner loop)
__device__ __forceinline__ uint32_t chain_saddr(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ int lds32(uint32_t a) {
  int v;
  asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts32(uint32_t a, int v) {
  asm volatile("st.shared.s32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
// hand-over words between the warps of the block
__device__ __forceinline__ int lds_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(chain_saddr(p)) : "memory");
  return v;
}
__device__ __forceinline__ void sts_release(int* p, int v) {
  asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(chain_saddr(p)), "r"(v) : "memory");
}
// Loads that observe what other SMs have written (they do not hit a stale L1 line) without
// ordering anything else: used to look at the router's flags and, once a flag has been seen
// set, to fetch the records it covers (the router wrote them before releasing the flag).
__device__ __forceinline__ uint32_t ld_relaxed_u32(const void* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u16(const void* p) {
  uint16_t v;
  asm volatile("ld.relaxed.gpu.global.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u8(const void* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u8 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld_relaxed_v2(const void* p) {
  uint2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ld_relaxed_v4(const void* p) {
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

struct ChainSlot {
  int32_t* fb;                // [E] fixed assignments of this call made before the group
  int32_t* db;                // [E] decisions of this call made before the group (by the chain)
  uint32_t* fm;               // [E] the group's masks of fixed tokens
  unsigned long long* ent;    // [32][CMAX] entries: load seen without decisions (all ones: no
                              //   candidate) | expert << 32 | cross-reference << 40 | token << 48
  uint8_t* ids;               // [32][CMAX] the group's ranked candidate ids (staging)
  uint32_t* out;              // [32] per entry: the chosen candidates (bit = lane)
  int* seq;                   // (group + 1) * 64 + entries once the slot is ready for the chain
  uint8_t* dl;                // [32] the group's decision tokens in order
};

template <int CMAX>
__device__ __forceinline__ ChainSlot chain_slot(unsigned char* slots, int slot, int E) {
  unsigned char* p = slots + (size_t)slot * k2_chain_slot_bytes(E, CMAX);
  ChainSlot s;
  s.fb = reinterpret_cast<int32_t*>(p);              p += align256(sizeof(int32_t) * E);
  s.db = reinterpret_cast<int32_t*>(p);              p += align256(sizeof(int32_t) * E);
  s.fm = reinterpret_cast<uint32_t*>(p);             p += align256(sizeof(int32_t) * E);
  s.ent = reinterpret_cast<unsigned long long*>(p);  p += (size_t)32 * CMAX * 8;
  s.ids = p;                                         p += (size_t)32 * CMAX;
  s.out = reinterpret_cast<uint32_t*>(p);            p += 128;
  s.seq = reinterpret_cast<int*>(p);
  s.dl = p + 32;
  return s;
}

// The whole layer.  smem: k2_chain_smem_bytes().  Lin (shared, [E]): the loads on entry; L_out
// (shared, [E]) receives the loads after the call; on return every thread of the block has
// passed a block barrier.  ready: the router's flags (one per router_rows tokens), or null if
// the records are already there.  fail(): called by one thread when a wait ran out; it raises
// the status and *gave_up.
template <int CMAX, typename FailFn>
__device__ __forceinline__ void k2_chain_layer(const RouteArgs& A, int layer, unsigned char* smem,
                                               int32_t* L_out, const int32_t* Lin, int* gave_up,
                                               const int* ready, int router_rows, FailFn fail) {
  constexpr int EPI = 32 / CMAX;   // entries built per pass of a helper warp
  constexpr int MW = kMaxExperts / 32;
  const int E = A.E, k = A.k, c = A.c, T = A.T;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  unsigned char* p = smem;
  int32_t* dcnt = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * E);
  int32_t* fcum = reinterpret_cast<int32_t*>(p);    p += align256(sizeof(int32_t) * E);
  int* fdone = reinterpret_cast<int*>(p);           // groups whose fixed counts are in fcum
  int* cons = fdone + 1;                            // groups the chain has finished
  p += 256;
  unsigned char* slots = p;

  unsigned char* ws = A.ws + (size_t)layer * A.ws_ls;
  const uint16_t* g_cs = reinterpret_cast<const uint16_t*>(ws + A.lay.cstar);
  const uint8_t* g_ids = ws + A.lay.cand_ids;
  const uint32_t* g_fm = reinterpret_cast<const uint32_t*>(ws + A.lay.fmask);
  uint32_t* g_selmask = reinterpret_cast<uint32_t*>(ws + A.lay.sel_mask);
  int32_t* g_base = reinterpret_cast<int32_t*>(ws + A.lay.grp_base);
  const int n_groups = A.lay.n_groups;

  for (int e = tid; e < E; e += blockDim.x) { dcnt[e] = 0; fcum[e] = 0; }
  if (tid == 0) { *fdone = 0; *cons = 0; }
  if (tid < kChainSlots) *chain_slot<CMAX>(slots, tid, E).seq = 0;
  __syncthreads();

  if (warp == 0) {
    // ---------------------------------------------------------------- the chain
    const bool mine = lane < CMAX;
    const int cl = lane & (CMAX - 1);
    const uint32_t dcnt_a = chain_saddr(dcnt);
    for (int g = 0; g < n_groups; ++g) {
      const ChainSlot S = chain_slot<CMAX>(slots, g % kChainSlots, E);
      int word = lds_acquire(S.seq);
      while ((word >> 6) != g + 1) {
        if (ld_volatile_shared(gave_up)) break;
        __nanosleep(20);
        word = lds_acquire(S.seq);
      }
      if ((word >> 6) != g + 1) break;   // the helpers gave up
      const int n = word & 63;
      // the decisions made before the group (the slot's helper adds the fixed assignments and
      // writes the group's base counts to global memory; the chain itself stores nothing there)
      {
        const uint32_t db_a = chain_saddr(S.db) + 4u * lane;
        int snap[MW];
#pragma unroll
        for (int q = 0; q < MW; ++q)
          if (32 * q < E) snap[q] = lds32(dcnt_a + 4u * (lane + 32 * q));
#pragma unroll
        for (int q = 0; q < MW; ++q)
          if (32 * q < E) sts32(db_a + 128u * q, snap[q]);
      }
      if (n > 0) {
        // entry 0: its counters are exact (every earlier increment has landed).  Entries are
        // read two ahead and their counters one ahead (past the end: the last entry again).
        // (word.x: load seen without decisions; word.y: expert | cross-reference << 8 | token << 16)
        const uint32_t ent_a = chain_saddr(S.ent) + 8u * (uint32_t)cl;
        const uint32_t out_a = chain_saddr(S.out);
        const uint32_t last_a = ent_a + (uint32_t)(n - 1) * (CMAX * 8u);
        uint2 w_c = lds64(ent_a), w_n = lds64(min(ent_a + CMAX * 8u, last_a));
        int d_c = lds32(dcnt_a + 4u * (w_c.y & 255u));
        unsigned chos_prev = 0;
        uint32_t next2 = ent_a + 2u * CMAX * 8u;
        for (int i = 0; i < n; ++i) {
          const uint2 w_f = lds64(min(next2, last_a));
          next2 += CMAX * 8u;
          const int d_n = lds32(dcnt_a + 4u * (w_n.y & 255u));   // before this entry's increments
          // Off the critical path: the key without the correction (all ones for a lane without
          // a candidate), and where the previous choice's bit for this lane's expert lands when
          // the ballot is rotated so that it sits at bit 5 (the unit of the load in the key).
          const uint32_t x_c = (w_c.y >> 8) & 255u;
          const bool has = mine && w_c.x != 0xffffffffu;
          const uint32_t key0 = has ? (((w_c.x + (uint32_t)d_c) << 5) | (uint32_t)cl) : 0xffffffffu;
          const uint32_t rot = (x_c - 5u) & 31u;
          const uint32_t unit = (has && x_c < 32u) ? 32u : 0u;
          // On it: previous ballot -> correction -> key -> all-pairs rank -> ballot.
          const uint32_t corr32 = __funnelshift_r(chos_prev, chos_prev, rot) & unit;
          const uint32_t key = key0 + corr32;
          int r0 = 0, r1 = 0;
#pragma unroll
          for (int j = 0; j < CMAX; j += 2) {
            r0 += __shfl_sync(0xffffffffu, key, j) < key ? 1 : 0;
            r1 += __shfl_sync(0xffffffffu, key, j + 1) < key ? 1 : 0;
          }
          // (a lane without a candidate ranks behind all c* > k candidates)
          const bool chosen = r0 + r1 < k;
          chos_prev = __ballot_sync(0xffffffffu, chosen);
          const int corr = (int)(corr32 >> 5);
          // the candidates of one token are distinct experts: a plain store per chosen lane
          if (chosen) sts32(dcnt_a + 4u * (w_c.y & 255u), d_c + (int)corr + 1);
          if (lane == 0) sts32(out_a + 4u * (uint32_t)i, (int)chos_prev);
          __syncwarp();
          w_c = w_n; w_n = w_f; d_c = d_n;
        }
      }
      __syncwarp();
      if (lane == 0) sts_release(cons, g + 1);
    }
  } else {
    // ---------------------------------------------------------------- the helpers
    const int hw = warp - 1;
    const ChainSlot S = chain_slot<CMAX>(slots, hw, E);
    // A look at the router's flags of group g without waiting: the raw flag value of this
    // lane's share (router tiles of 16 tokens: two flags per group), judged a trip later.
    auto look = [&](int g) -> int {
      if (!ready || g >= n_groups) return ready ? 0 : 1;
      const int t0 = g * 32, rt_last = (min(T, t0 + 32) - 1) / router_rows;
      const int rt = min(t0 / router_rows + (router_rows < 32 ? (lane & 1) : 0), rt_last);
      return (int)ld_relaxed_u32(ready + rt);
    };
    uint32_t mw[MW];      // the group's masks of experts lane, lane + 32, ...
    int cs = 0;           // c* of token lane
    uint4 idv = make_uint4(0, 0, 0, 0);   // its first 16 ranked ids (c <= 16)
    auto load_group = [&](int g) {
      const int t = g * 32 + lane;
      cs = t < T ? (int)ld_relaxed_u16(g_cs + t) : 0;
#pragma unroll
      for (int q = 0; q < MW; ++q)
        mw[q] = lane + 32 * q < E ? ld_relaxed_u32(g_fm + (size_t)g * E + lane + 32 * q) : 0u;
      if (t < T && c <= 16) {
        const uint8_t* src = g_ids + (size_t)t * c;
        if (c == 16) idv = ld_relaxed_v4(src);
        else if (c == 8) { const uint2 v = ld_relaxed_v2(src); idv.x = v.x; idv.y = v.y; }
        else if (c == 4) idv.x = ld_relaxed_u32(src);
        else {
          uint32_t wv[4] = {0, 0, 0, 0};
          for (int r = 0; r < c; ++r) wv[r >> 2] |= ld_relaxed_u8(src + r) << (8 * (r & 3));
          idv = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
    };
    // What the chain left in the slot for group g goes to global memory: the decision tokens'
    // choices and the group's base counts (fixed assignments + decisions made before it).
    auto flush = [&](int g, int n) {
      if (lane < n) {
        const int tok = (int)(S.ent[lane * CMAX] >> 48) & 31;
        g_selmask[(size_t)g * 32 + tok] = S.out[lane];
      }
      int32_t* gb = g_base + (size_t)g * E;
      for (int e = lane; e < E; e += 32) gb[e] = S.fb[e] + S.db[e];
      __syncwarp();
    };
    bool ok = true;
    bool have = false;        // the records of this trip's group are already in registers
    int fv_next = look(hw + kChainSlots);   // flags of the next trip's group, judged next trip
    int n_prev = 0;           // entries of the group this slot held before
    for (int g = hw; g < n_groups; g += kChainSlots) {
      // the slot's previous group must have been consumed; its choices go to global memory
      if (g >= kChainSlots) {
        const long long start = clock64();
        unsigned ns = 20;   // polls grow rarer: the chain shares this SM's shared-memory pipe
        while (lds_acquire(cons) < g - kChainSlots + 1) {
          if (ld_volatile_shared(gave_up) || clock64() - start > A.wait_cycles) { ok = false; break; }
          __nanosleep(ns);
          ns = min(ns * 2u, 400u);
        }
        if (!ok) break;
        flush(g - kChainSlots, n_prev);
      }
      if (!have) {
        if (ready) {
          const int t0 = g * 32;
          if (!k2_wait_ready(ready, router_rows, t0, min(T, t0 + 32) - 1, A.wait_cycles)) {
            ok = false;
            break;
          }
        }
        load_group(g);
      }
      // masks and ids into the slot, per-expert counts of the group
      int cnt[MW];
#pragma unroll
      for (int q = 0; q < MW; ++q) {
        cnt[q] = __popc(mw[q]);
        if (lane + 32 * q < E) S.fm[lane + 32 * q] = mw[q];
      }
      if (c <= 16) {
        if (CMAX == 16) *reinterpret_cast<uint4*>(S.ids + lane * 16) = idv;
        else if (CMAX == 8) *reinterpret_cast<uint2*>(S.ids + lane * 8) = make_uint2(idv.x, idv.y);
        else *reinterpret_cast<uint32_t*>(S.ids + lane * 4) = idv.x;
      } else {
        const int t = g * 32 + lane;
        if (t < T)
          for (int r = 0; r < c; ++r)
            S.ids[lane * CMAX + r] = (uint8_t)ld_relaxed_u8(g_ids + (size_t)t * c + r);
      }
      const int my_cs = cs;
      // look ahead: if the next trip's group was seen published, request its records now (the
      // registers are free again); and take a look at the flags of the trip after that
      const int g1 = g + kChainSlots;
      have = g1 < n_groups && __all_sync(0xffffffffu, fv_next > 0);
      if (have) load_group(g1);
      fv_next = look(g1 + kChainSlots);
      // the running count of fixed assignments: taken over from the group before, passed on
      {
        const long long start = clock64();
        while (lds_acquire(fdone) < g) {
          if (ld_volatile_shared(gave_up) || clock64() - start > A.wait_cycles) { ok = false; break; }
          __nanosleep(20);
        }
        if (!ok) break;
        {
          // all loads first, then the stores (explicit shared-memory accesses: nothing here
          // waits for a store to land before the next load)
          const uint32_t fc_a = chain_saddr(fcum) + 4u * lane, fb_a = chain_saddr(S.fb) + 4u * lane;
          int f[MW];
#pragma unroll
          for (int q = 0; q < MW; ++q)
            if (32 * q < E) f[q] = lds32(fc_a + 128u * q);
#pragma unroll
          for (int q = 0; q < MW; ++q)
            if (32 * q < E) {
              sts32(fc_a + 128u * q, f[q] + cnt[q]);
              sts32(fb_a + 128u * q, f[q]);
            }
        }
        __syncwarp();
        if (lane == 0) sts_release(fdone, g + 1);
      }
      // one entry per decision token, CMAX lanes each
      const unsigned dmask = __ballot_sync(0xffffffffu, my_cs > k);
      const int n = __popc(dmask);
      if (my_cs > k) S.dl[__popc(dmask & ((1u << lane) - 1u))] = (uint8_t)lane;
      __syncwarp();
      const int r = lane & (CMAX - 1);
      for (int i0 = 0; i0 < n; i0 += EPI) {
        const int i = min(i0 + lane / CMAX, n - 1);   // (lanes past the end redo the last entry)
        const int tokl = S.dl[i];
        const int cs_i = __shfl_sync(0xffffffffu, my_cs, tokl);
        const int e = S.ids[tokl * CMAX + r];
        const bool has = r < cs_i;
        const uint32_t seen =
            has ? (uint32_t)(Lin[e] + S.fb[e] + __popc(S.fm[e] & ((1u << tokl) - 1u))) : 0xffffffffu;
        // the lane of the previous entry (same group) that holds the same expert
        uint32_t x = 32;
        if (i > 0) {
          const uint32_t* prev = reinterpret_cast<const uint32_t*>(S.ids + (int)S.dl[i - 1] * CMAX);
          const uint32_t pat = (uint32_t)e * 0x01010101u;
          uint32_t pw[CMAX / 4];
          if constexpr (CMAX >= 16) {
#pragma unroll
            for (int q = 0; q < CMAX / 16; ++q) {
              const uint4 v = reinterpret_cast<const uint4*>(prev)[q];
              pw[4 * q] = v.x; pw[4 * q + 1] = v.y; pw[4 * q + 2] = v.z; pw[4 * q + 3] = v.w;
            }
          } else {
#pragma unroll
            for (int q = 0; q < CMAX / 4; ++q) pw[q] = prev[q];
          }
#pragma unroll
          for (int q = CMAX / 4 - 1; q >= 0; --q) {
            const uint32_t m = __vcmpeq4(pw[q], pat);     // 0xff in every byte that matches
            if (m) x = 4 * q + ((__ffs(m) - 1) >> 3);     // the lowest lane wins
          }
        }
        S.ent[i * CMAX + r] = (unsigned long long)seen | ((unsigned long long)e << 32) |
                              ((unsigned long long)x << 40) | ((unsigned long long)tokl << 48);
      }
      __syncwarp();
      if (lane == 0) sts_release(S.seq, (g + 1) * 64 + n);
      n_prev = n;
    }
    // the choices of the slot's last group
    if (ok && n_groups > hw) {
      const int g_last = hw + ((n_groups - 1 - hw) / kChainSlots) * kChainSlots;
      const long long start = clock64();
      while (lds_acquire(cons) < g_last + 1) {
        if (ld_volatile_shared(gave_up) || clock64() - start > A.wait_cycles) { ok = false; break; }
        __nanosleep(500);
      }
      if (ok) flush(g_last, n_prev);
    }
    if (!ok && lane == 0 && !ld_volatile_shared(gave_up)) fail();
  }
  __syncthreads();
  for (int e = tid; e < E; e += blockDim.x) L_out[e] = Lin[e] + fcum[e] + dcnt[e];
  __syncthreads();
}

}  // namespace laser
