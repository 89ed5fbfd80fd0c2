// Shared device helpers and the per-layer argument block of the LASER routing kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace laser {

constexpr int kMaxLayersPerLaunch = 64;
constexpr int kMaxExperts = 256;

// Scratch carved from the caller's workspace for one layer.  Offsets in bytes.
struct WorkspaceLayout {
  size_t cstar;        // uint16 [T]        0 = top-k branch, else c*
  size_t cand_ids;     // uint8  [T, c]     ranking pi(0..c-1)
  size_t cand_scores;  // float  [T, c]     s_pi(j)
  size_t sel_rank;     // uint8  [T, k]     rank positions chosen by the load-aware scan
  size_t grp_base;     // int32  [n_groups, E]  per-expert count of this call's assignments made
                       //                   before the group (load at group start minus L_in)
  size_t fmask;        // uint32 [n_groups, E]  (E > 32 only) bit i: token i of the group has no
                       //                   load-dependent choice and goes to this expert; router
                       //                   tiles of 16 tokens write their 16-bit half
  size_t sel_mask;     // uint32 [T]  (E > 32 only) the chosen candidates of a decision token as a
                       //                   bit mask over score ranks, where the selection ran as
                       //                   the pipeline of k2_chain.cuh (mode word = 1)
  size_t ready;        // int32  [ceil(T/16)+2] router tiles published to the selection role
                       //                   (1 = records written, -1 = the tile gave up); the last
                       //                   word is the layer's abort word: non-zero once a wait ran
                       //                   out, and then no later stage reads the layer's scratch;
                       //                   the word after it is the mode word: 1 if the decision
                       //                   tokens' choices are in sel_mask, 0 if in sel_rank
  size_t total;        // bytes per layer, multiple of 256
  int n_groups;        // ceil(T / 32): the ordered selection and the dispatch work on groups
                       // of 32 consecutive tokens
};

__host__ __device__ inline size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

inline WorkspaceLayout make_layout(int T, int E, int k, int c) {
  WorkspaceLayout w;
  size_t off = 0;
  w.n_groups = (T + 31) / 32;
  w.cstar = off;        off = align256(off + sizeof(uint16_t) * (size_t)T);
  w.cand_ids = off;     off = align256(off + (size_t)T * c);
  w.cand_scores = off;  off = align256(off + sizeof(float) * (size_t)T * c);
  w.sel_rank = off;     off = align256(off + (size_t)T * k);
  w.grp_base = off;     off = align256(off + sizeof(int32_t) * (size_t)w.n_groups * E);
  w.fmask = off;        off = align256(off + (E > 32 ? sizeof(uint32_t) * (size_t)w.n_groups * E : 0));
  w.sel_mask = off;     off = align256(off + (E > 32 ? sizeof(uint32_t) * (size_t)T : 0));
  w.ready = off;        off = align256(off + sizeof(int32_t) * (size_t)((T + 15) / 16 + 2));
  w.total = off;
  return w;
}

// Kernel-side view of one batched call: layer l uses base + l * stride of every array.
struct RouteArgs {
  const uint16_t* hidden;  long long hidden_ls;   // elements
  const uint16_t* wg;      long long wg_ls;
  const float* bias;       // [L, E] or null
  int32_t* loads;          // [L, E]
  const int32_t* e2b;      // [E] or null
  int32_t* bin_loads;      // [L, B] or null
  int fresh;               // the counters start from zero whatever loads / bin_loads hold
  int32_t* expert_ids;     // [L, T, k]
  float* weights;          // [L, T, k]
  int32_t* offsets;        // [L, E+1]
  int32_t* perm;           // [L, T*k]
  float* logits_out;       // [L, T, E] or null
  int32_t* status;         // device status word or null
  unsigned char* ws;       size_t ws_ls;          // bytes
  WorkspaceLayout lay;
  int T, d, E, k, c, n_bins, renorm;
  int trim_random;         // 1 = RANDOM trimming of the pool (Philox draws), 0 = TOP
  unsigned long long seed; // RANDOM trimming: generator key
  int G;                   // load-update granularity: 1 = after every token (the rule);
                           // 0 or a multiple of 32 = relaxed variant (loads seen refreshed
                           // every G tokens, 0 = once per call)
  long long ld_h, ld_w;
  int fuse_dispatch;       // 1 = the selection block also runs the dispatch of its layer (calls
                           //     of a few groups), and no dispatch kernel is launched
  int layer0;              // first layer of this launch
  int cluster_tiles;       // > 0: the layer's router tiles and its selection block form one
                           //      thread-block cluster (that many tiles + 1) and meet at the
                           //      cluster barrier; no ready flags are used.  0: ready flags
  long long wait_cycles;   // limit of the selection's waits for the router, in clock cycles
  int withhold_tile;       // test hook: the router tile with this index publishes no flag (-1: none)
  float eps_high[kMaxLayersPerLaunch];
  float t_fix[kMaxLayersPerLaunch];
};

// The layer's abort word (see WorkspaceLayout::ready).
__host__ __device__ inline size_t abort_word_index(int T) { return (size_t)((T + 15) / 16); }
__host__ __device__ inline size_t mode_word_index(int T) { return abort_word_index(T) + 1; }

// Rank position (in the score ranking) of slot j of token t as the selection left it:
// tokens with c* > k were decided by the load-aware scan (sel_rank), all others keep their
// k best in score order.
__device__ __forceinline__ int pair_rank(const uint16_t* cstar, const uint8_t* sel_rank, int k,
                                         long long t, int j) {
  return cstar[t] > k ? sel_rank[t * k + j] : j;
}

// fp32 exponential for y <= 0 with a fixed sequence of correctly rounded operations:
//   y < -80 -> 0;  n = rint(y*log2e);  r = y - n*ln2 (two fma steps);
//   degree-7 Taylor polynomial in Horner form;  result = p * 2^n.
__device__ __forceinline__ float exp32(float y) {
  float n = rintf(__fmul_rn(y, __uint_as_float(0x3FB8AA3Bu)));
  float r = __fmaf_rn(n, -__uint_as_float(0x3F317200u), y);
  r = __fmaf_rn(n, -__uint_as_float(0x35BFBE8Eu), r);
  float p = __uint_as_float(0x39500D01u);
  p = __fmaf_rn(p, r, __uint_as_float(0x3AB60B61u));
  p = __fmaf_rn(p, r, __uint_as_float(0x3C088889u));
  p = __fmaf_rn(p, r, __uint_as_float(0x3D2AAAABu));
  p = __fmaf_rn(p, r, __uint_as_float(0x3E2AAAABu));
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  int ni = __float2int_rn(n);                       // in [-116, 0] for y >= -80
  const float v = __fmul_rn(p, __int_as_float((ni + 127) << 23));
  return y < -80.0f ? 0.0f : v;                     // a select, so that calls interleave
}

}  // namespace laser
