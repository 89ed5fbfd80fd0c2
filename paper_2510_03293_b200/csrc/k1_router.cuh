// K1: router contraction x = h.W_g^T + b fused with the per-token score epilogue
// (softmax, ranking of the c best, top-k mass test, candidate count c*).
//
// Streaming design for small/medium E: each warp owns MT*16 token rows and walks the hidden
// dimension in chunks of 32 elements.  A thread reads 16 contiguous bytes of a row straight
// from global memory into the A fragment of two m16n8k16 bf16 MMAs (the contraction index is
// permuted identically for A and B, which a dot product allows), so hidden states go
// HBM -> registers -> tensor core with no shared-memory staging.  W_g is small and stays in
// L1/L2.  Accumulators are fp32.
#pragma once
#include "laser_common.cuh"

namespace laser {

// 16 bytes of hidden state, read once: not kept in L1, and fetched from memory 256 bytes at a
// time (a hint: the rest of the 256 bytes is asked for by the neighbouring loads anyway).
__device__ __forceinline__ uint4 ldg_stream(const uint16_t* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Per-token epilogue run by one thread on a row of fp32 logits in shared memory.
//   ranking pi by (logit desc, index asc); e_i = exp32(x_i - x_max);
//   Z = eight interleaved running sums combined pairwise; s = e / Z;
//   M_k = s_pi(0) + ... + s_pi(k-1) left to right; top-k branch iff M_k >= eps_high;
//   otherwise c* = max(k, #{j < c : s_pi(j) >= t_fix * s_pi(0)}).
// Writes the record (c*, ranked ids, ranked scores) for the load-aware scan and the dispatch,
// which derives every token's final ids and combine weights from it.
// fm (shared memory, may be null): per-expert masks of the token's group; a token without a
// load-dependent choice (top-k branch or c* == k) sets its bit for each of its k best.
__device__ __forceinline__ void token_epilogue(const float* __restrict__ x, int E, int k, int c,
                                               float eps_high, float t_fix, int renorm,
                                               uint16_t* cstar, uint8_t* cand_ids,
                                               float* cand_scores, uint32_t* fm = nullptr,
                                               uint32_t bit = 0) {
  float xmax = x[0];
  for (int i = 1; i < E; ++i) xmax = fmaxf(xmax, x[i]);

  float a[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = 0.0f;
  for (int i0 = 0; i0 < E; i0 += 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (i0 + j < E) a[j] = __fadd_rn(a[j], exp32(__fsub_rn(x[i0 + j], xmax)));
    }
  }
  const float Z = __fadd_rn(__fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3])),
                            __fadd_rn(__fadd_rn(a[4], a[5]), __fadd_rn(a[6], a[7])));

  float prev_x = __int_as_float(0x7f800000);  // +inf
  int prev_i = -1;
  float Mk = 0.0f, thr = 0.0f;
  int mprime = 0;
  for (int r = 0; r < c; ++r) {
    float bx = 0.0f;
    int bi = -1;
    for (int i = 0; i < E; ++i) {
      const float xi = x[i];
      const bool after_prev = (xi < prev_x) || (xi == prev_x && i > prev_i);
      if (after_prev && (bi < 0 || xi > bx)) { bx = xi; bi = i; }
    }
    const float s = __fdiv_rn(exp32(__fsub_rn(bx, xmax)), Z);
    if (r == 0) { thr = __fmul_rn(t_fix, s); Mk = s; }
    else if (r < k) Mk = __fadd_rn(Mk, s);
    if (s >= thr) ++mprime;
    cand_ids[r] = (uint8_t)bi;
    cand_scores[r] = s;
    prev_x = bx;
    prev_i = bi;
  }
  const bool top_k_branch = (Mk >= eps_high);
  *cstar = top_k_branch ? (uint16_t)0 : (uint16_t)max(k, mprime);
  if (fm && (top_k_branch || mprime <= k))
    for (int j = 0; j < k; ++j) atomicOr(&fm[cand_ids[j]], bit);   // (reads its own stores)
}

// ---- RANDOM trimming (Algorithm 1, mode RANDOM) ---------------------------------------------
// Philox4x32-10 (Salmon et al., SC 2011): ten rounds of
//   (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)),
// the key advancing by the Weyl constants between rounds.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t n0 = __umulhi(M1, c2) ^ c1 ^ k0, n1 = M1 * c2;
    const uint32_t n2 = __umulhi(M0, c0) ^ c3 ^ k1, n3 = M0 * c0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Per-token epilogue with RANDOM trimming, one thread on a row of logits in shared memory.
// Softmax, ranking and the top-k mass test are those of token_epilogue.  On the expanded branch
//   pool  = ranking prefix of length m = max(k, #{i : s_i >= t_fix * s_pi(0)}) over all E,
//   c*    = min(c, m); if c* < m a partial Fisher-Yates shuffle draws the sample:
//           for i < c*:  j = i + u_i mod (m - i), swap  (u_i = word i % 4 of the Philox block
//           with key = seed and counter = (token, layer, i / 4, 0)),
//   the record lists the c* sampled experts in score-rank order.
// Not a fast path: it ranks up to E experts round by round and keeps two byte arrays in local
// memory.
static __device__ __noinline__ void token_epilogue_random(const float* row, int E, int k, int c,
                                                   float eps_high, float t_fix, int renorm,
                                                   unsigned long long seed, int layer, long long t,
                                                   uint16_t* cstar, uint8_t* cand_ids,
                                                   float* cand_scores, uint32_t* fm = nullptr,
                                                   uint32_t bit = 0) {
  float xmax = row[0];
  for (int i = 1; i < E; ++i) xmax = fmaxf(xmax, row[i]);
  float a[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = 0.0f;
  for (int i0 = 0; i0 < E; i0 += 8) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (i0 + j < E) a[j] = __fadd_rn(a[j], exp32(__fsub_rn(row[i0 + j], xmax)));
  }
  const float Z = __fadd_rn(__fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3])),
                            __fadd_rn(__fadd_rn(a[4], a[5]), __fadd_rn(a[6], a[7])));
  const float thr = __fmul_rn(t_fix, __fdiv_rn(exp32(0.0f), Z));   // s of the best expert
  int m = 0;
  for (int i = 0; i < E; ++i)
    if (__fdiv_rn(exp32(__fsub_rn(row[i], xmax)), Z) >= thr) ++m;
  if (m < k) m = k;

  uint8_t R[kMaxExperts];   // R[r]: expert of rank r
  uint8_t P[kMaxExperts];   // rank positions, shuffled
  float prev_x = __int_as_float(0x7f800000);  // +inf
  int prev_i = -1;
  float Mk = 0.0f;
  int need = k;
  for (int r = 0; r < need; ++r) {
    float bx = 0.0f;
    int bi = -1;
    for (int i = 0; i < E; ++i) {
      const float xi = row[i];
      const bool after_prev = (xi < prev_x) || (xi == prev_x && i > prev_i);
      if (after_prev && (bi < 0 || xi > bx)) { bx = xi; bi = i; }
    }
    R[r] = (uint8_t)bi;
    if (r < k) {
      const float s = __fdiv_rn(exp32(__fsub_rn(bx, xmax)), Z);
      Mk = r == 0 ? s : __fadd_rn(Mk, s);
      cand_ids[r] = (uint8_t)bi;   // the top-k branch's record: the selection and the dispatch
      cand_scores[r] = s;          // read the k best from here (overwritten by a sample)
      if (r == k - 1 && !(Mk >= eps_high)) need = m;   // expanded: rank the whole pool
    }
    prev_x = bx;
    prev_i = bi;
  }
  if (Mk >= eps_high) {
    *cstar = 0;
    if (fm)
      for (int j = 0; j < k; ++j) atomicOr(&fm[cand_ids[j]], bit);
    return;
  }
  const int cs = c < m ? c : m;
  for (int i = 0; i < m; ++i) P[i] = (uint8_t)i;
  if (cs < m) {
    uint32_t blk[4];
    for (int i = 0; i < cs; ++i) {
      if ((i & 3) == 0)
        philox4x32_10((uint32_t)t, (uint32_t)layer, (uint32_t)(i >> 2), 0u, (uint32_t)seed,
                      (uint32_t)(seed >> 32), blk);
      const uint32_t u = (i & 3) == 0 ? blk[0] : ((i & 3) == 1 ? blk[1] : ((i & 3) == 2 ? blk[2] : blk[3]));
      const int j = i + (int)(u % (uint32_t)(m - i));
      const uint8_t tmp = P[i]; P[i] = P[j]; P[j] = tmp;
    }
  }
  for (int i = 1; i < cs; ++i) {   // the sample in score-rank order
    const uint8_t v = P[i];
    int pos = i;
    while (pos > 0 && P[pos - 1] > v) { P[pos] = P[pos - 1]; --pos; }
    P[pos] = v;
  }
  for (int j = 0; j < cs; ++j) {
    const int e = R[P[j]];
    cand_ids[j] = (uint8_t)e;
    cand_scores[j] = __fdiv_rn(exp32(__fsub_rn(row[e], xmax)), Z);
  }
  *cstar = (uint16_t)cs;
  if (fm && cs <= k)   // a sample of exactly k experts leaves nothing to decide
    for (int j = 0; j < k; ++j) atomicOr(&fm[cand_ids[j]], bit);
}

// ---- score epilogue with sorting networks (one thread per token) ---------------------------
// Descending bitonic sort of N (power of two) registers.
template <int N>
__device__ __forceinline__ void sort_desc(uint32_t (&a)[N]) {
#pragma unroll
  for (int size = 2; size <= N; size <<= 1) {
#pragma unroll
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const int j = i ^ stride;
        if (j > i) {
          const uint32_t lo = min(a[i], a[j]), hi = max(a[i], a[j]);
          const bool down = (i & size) == 0;
          a[i] = down ? hi : lo;
          a[j] = down ? lo : hi;
        }
      }
    }
  }
}
// Sorts a bitonic sequence of N registers into descending order.
template <int N>
__device__ __forceinline__ void bitonic_merge_desc(uint32_t (&a)[N]) {
#pragma unroll
  for (int stride = N >> 1; stride > 0; stride >>= 1) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const int j = i ^ stride;
      if (j > i) {
        const uint32_t lo = min(a[i], a[j]), hi = max(a[i], a[j]);
        a[i] = hi;
        a[j] = lo;
      }
    }
  }
}

// Per-token score epilogue by one thread on a row of fp32 logits in shared memory, for
// 32 < E <= N (N = 64 or 128) and c <= CL.  Same results as token_epilogue, found faster:
// every logit becomes a 32-bit key  (order-preserving bits of x with the low log2(N) bits
// replaced by N-1-index), groups of CL keys are sorted by a bitonic network and merged into
// the running CL best (element-wise maximum against the reversed list, then a bitonic merge).
// Dropping the low bits of x can only misorder two logits that agree in all kept bits; the
// ranking is therefore accepted only if the kept bits of neighbouring entries of the best
// c + 1 differ strictly (then x itself differs strictly in the same direction, and nothing
// outside the list can belong inside); otherwise the token is redone by token_epilogue.
// The softmax is the one of token_epilogue, operation by operation.
template <int N, int CL>
__device__ __forceinline__ void token_epilogue_sorted(const float* __restrict__ row, int E, int k,
                                                      int c, float eps_high, float t_fix,
                                                      int renorm, uint16_t* cstar,
                                                      uint8_t* cand_ids, float* cand_scores,
                                                      uint32_t* fm = nullptr, uint32_t bit = 0) {
  constexpr uint32_t IDX = N - 1;
  constexpr int SH = N == 64 ? 6 : 7;
  static_assert(N == 64 || N == 128, "index bits");
  // The row has N >= E readable columns (those from E on are ignored), so that every group of
  // CL columns is loaded and exponentiated without a branch and the calls interleave.
  float xmax;
  {
    float m[4] = {row[0], row[0], row[0], row[0]};
    int i = 0;
    for (; i + 4 <= E; i += 4) {
#pragma unroll
      for (int q = 0; q < 4; ++q) m[q] = fmaxf(m[q], row[i + q]);
    }
    for (; i < E; ++i) m[0] = fmaxf(m[0], row[i]);
    xmax = fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
  }

  float a[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) a[j] = 0.0f;
  uint32_t R[CL];      // the CL best keys so far, descending
  uint32_t dm = 0;     // the best key that was dropped from R
#pragma unroll
  for (int i = 0; i < CL; ++i) R[i] = 0;
#pragma unroll 1
  for (int g0 = 0; g0 < E; g0 += CL) {
    uint32_t B[CL];
    float xv[CL], ev[CL];
#pragma unroll
    for (int i = 0; i < CL; ++i) xv[i] = row[g0 + i];   // g0 + i < N
#pragma unroll
    for (int i = 0; i < CL; ++i) ev[i] = exp32(__fsub_rn(xv[i], xmax));
#pragma unroll
    for (int i = 0; i < CL; ++i) {
      const int e = g0 + i;
      const bool in = e < E;
      a[i & 7] = __fadd_rn(a[i & 7], in ? ev[i] : 0.0f);   // a >= +0: adding +0 changes nothing
      const uint32_t u = __float_as_uint(xv[i]);
      const uint32_t o = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
      B[i] = in ? ((o & ~IDX) | (IDX - (uint32_t)e)) : 0u;
    }
    sort_desc<CL>(B);
    if (g0 == 0) {
#pragma unroll
      for (int i = 0; i < CL; ++i) R[i] = B[i];
    } else {
#pragma unroll
      for (int i = 0; i < CL; ++i) {
        const uint32_t p = R[i], q = B[CL - 1 - i];
        R[i] = max(p, q);
        dm = max(dm, min(p, q));
      }
      bitonic_merge_desc<CL>(R);
    }
  }
  const float Z = __fadd_rn(__fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3])),
                            __fadd_rn(__fadd_rn(a[4], a[5]), __fadd_rn(a[6], a[7])));
  bool exact = true;
#pragma unroll
  for (int i = 0; i < CL; ++i) {
    if (i < c) {
      const uint32_t next = (i + 1 < CL) ? R[(i + 1 < CL) ? i + 1 : i] : dm;
      exact = exact && ((R[i] >> SH) > (next >> SH));
    }
  }
  if (!exact) {
    token_epilogue(row, E, k, c, eps_high, t_fix, renorm, cstar, cand_ids, cand_scores, fm, bit);
    return;
  }
  float Mk = 0.0f, thr = 0.0f;
  int mprime = 0;
  float sv[CL];   // scores of all CL listed ranks at once (those from c on are not used)
#pragma unroll
  for (int r = 0; r < CL; ++r)
    sv[r] = __fdiv_rn(exp32(__fsub_rn(row[IDX - (R[r] & IDX)], xmax)), Z);
#pragma unroll
  for (int r = 0; r < CL; ++r) {
    if (r < c) {
      const float s = sv[r];
      if (r == 0) { thr = __fmul_rn(t_fix, s); Mk = s; }
      else if (r < k) Mk = __fadd_rn(Mk, s);
      if (s >= thr) ++mprime;
    }
  }
  const bool top_k_branch = (Mk >= eps_high);
  *cstar = top_k_branch ? (uint16_t)0 : (uint16_t)max(k, mprime);
  if (fm && (top_k_branch || mprime <= k)) {
#pragma unroll
    for (int r = 0; r < CL; ++r)
      if (r < k) atomicOr(&fm[IDX - (R[r] & IDX)], bit);
  }
  // Records out (the final ids and weights of every token are written by the dispatch).  With
  // c = 8 a token's record is written with 8- and 16-byte stores: the stores of a warp go to 32
  // different sectors each, so their number is what costs.
  if constexpr (CL == 8) {
    // (the scratch records are 8 and 32 bytes per token in a 256-byte aligned workspace)
    if (c == 8) {
      uint32_t lo = 0, hi = 0;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        lo |= (IDX - (R[r] & IDX)) << (8 * r);
        hi |= (IDX - (R[r + 4] & IDX)) << (8 * r);
      }
      *reinterpret_cast<uint2*>(cand_ids) = make_uint2(lo, hi);
      *reinterpret_cast<float4*>(cand_scores) = make_float4(sv[0], sv[1], sv[2], sv[3]);
      *reinterpret_cast<float4*>(cand_scores + 4) = make_float4(sv[4], sv[5], sv[6], sv[7]);
      return;
    }
  }
#pragma unroll
  for (int r = 0; r < CL; ++r) {
    if (r < c) {
      const int bi = (int)(IDX - (R[r] & IDX));
      cand_ids[r] = (uint8_t)bi;
      cand_scores[r] = sv[r];
    }
  }
}

// Score epilogue of 4 tokens by one warp, 8 lanes per token (same arithmetic, operation by
// operation, as token_epilogue on a shared-memory row):
//   ranking pi by (logit desc, index asc);  e_i = exp32(x_i - x_max);
//   Z = eight interleaved running sums a_j = sum_{i = j mod 8, ascending} e_i combined as
//       ((a0+a1)+(a2+a3))+((a4+a5)+(a6+a7));  s = e / Z;  M_k left to right;
//   top-k branch iff M_k >= eps_high;  otherwise c* = max(k, #{j < c : s_pi(j) >= t_fix*s_pi(0)}).
// row: the token's logits in shared memory (nullptr-safe only through write = false with a
// valid row).  Lane j of the group owns experts 8m + j.  All 32 lanes must call.
template <int N>
__device__ __forceinline__ void token_epilogue_lanes8(const float* row, int j, int E, int k, int c,
                                                      float eps_high, float t_fix, int renorm,
                                                      bool write, uint16_t* cstar,
                                                      uint8_t* cand_ids, float* cand_scores,
                                                      uint32_t* fm = nullptr, uint32_t bit = 0) {
  constexpr int EPL = N / 8;
  const float ninf = __int_as_float(0xff800000);
  float x[EPL];
  float xmax = ninf;
#pragma unroll
  for (int m = 0; m < EPL; ++m) {
    const int i = 8 * m + j;
    x[m] = i < E ? row[i] : ninf;
    xmax = fmaxf(xmax, x[m]);
  }
#pragma unroll
  for (int s = 1; s < 8; s <<= 1) xmax = fmaxf(xmax, __shfl_xor_sync(0xffffffffu, xmax, s));
  float a = 0.0f;
#pragma unroll
  for (int m = 0; m < EPL; ++m)
    if (8 * m + j < E) a = __fadd_rn(a, exp32(__fsub_rn(x[m], xmax)));
  float Z = a;
#pragma unroll
  for (int s = 1; s < 8; s <<= 1) Z = __fadd_rn(Z, __shfl_xor_sync(0xffffffffu, Z, s));

  float prev_x = __int_as_float(0x7f800000);  // +inf
  int prev_i = -1;
  if (c > 32) {
    // wide candidate lists (rare): score every rank as it is found
    float Mk = 0.0f, thr = 0.0f;
    int mprime = 0;
#pragma unroll 1
    for (int r = 0; r < c; ++r) {
      float bx = ninf;
      int bi = 0x7fffffff;
#pragma unroll
      for (int m = 0; m < EPL; ++m) {
        const int i = 8 * m + j;
        const float xi = x[m];
        const bool after_prev = (xi < prev_x) || (xi == prev_x && i > prev_i);
        if (i < E && after_prev && xi > bx) { bx = xi; bi = i; }
      }
#pragma unroll
      for (int s = 1; s < 8; s <<= 1) {
        const float ox = __shfl_xor_sync(0xffffffffu, bx, s);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
        if (ox > bx || (ox == bx && oi < bi)) { bx = ox; bi = oi; }
      }
      const float sr = __fdiv_rn(exp32(__fsub_rn(bx, xmax)), Z);
      if (r == 0) { thr = __fmul_rn(t_fix, sr); Mk = sr; }
      else if (r < k) Mk = __fadd_rn(Mk, sr);
      if (sr >= thr) ++mprime;
      if (write && j == 0) {
        cand_ids[r] = (uint8_t)bi;
        cand_scores[r] = sr;
      }
      prev_x = bx;
      prev_i = bi;
    }
    if (!write || j != 0) return;
    const bool top_k_branch = (Mk >= eps_high);
    *cstar = top_k_branch ? (uint16_t)0 : (uint16_t)max(k, mprime);
    if (fm && (top_k_branch || mprime <= k))
      for (int q = 0; q < k; ++q) atomicOr(&fm[cand_ids[q]], bit);
    return;
  }
  // ranking: c rounds of "best remaining" (local scan, then a 3-step butterfly over the group);
  // lane j keeps the results of ranks j, j+8, j+16, j+24
  float kx[4] = {ninf, ninf, ninf, ninf};
  int ki[4] = {0, 0, 0, 0};
#pragma unroll 1
  for (int r = 0; r < c; ++r) {
    float bx = ninf;
    int bi = 0x7fffffff;
#pragma unroll
    for (int m = 0; m < EPL; ++m) {
      const int i = 8 * m + j;
      const float xi = x[m];
      const bool after_prev = (xi < prev_x) || (xi == prev_x && i > prev_i);
      if (i < E && after_prev && xi > bx) { bx = xi; bi = i; }
    }
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) {
      const float ox = __shfl_xor_sync(0xffffffffu, bx, s);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
      if (ox > bx || (ox == bx && oi < bi)) { bx = ox; bi = oi; }
    }
    if ((r & 7) == j) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if ((r >> 3) == q) { kx[q] = bx; ki[q] = bi; }
    }
    prev_x = bx;
    prev_i = bi;
  }
  // scores of this lane's ranks
  float sc[4];
#pragma unroll
  for (int q = 0; q < 4; ++q)
    sc[q] = (8 * q + j < c) ? __fdiv_rn(exp32(__fsub_rn(kx[q], xmax)), Z) : 0.0f;
  // M_k = s_pi(0) + ... + s_pi(k-1), left to right; rank r lives in lane r % 8, slot r / 8
  const int gbase = (threadIdx.x & 31) & ~7;
  float Mk = 0.0f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (8 * q < k) {   // uniform over the warp
#pragma unroll
      for (int l = 0; l < 8; ++l) {
        const float v = __shfl_sync(0xffffffffu, sc[q], gbase + l);
        const int r = 8 * q + l;
        if (r < k) Mk = r == 0 ? v : __fadd_rn(Mk, v);
      }
    }
  }
  const float s0 = __shfl_sync(0xffffffffu, sc[0], gbase);
  const float thr = __fmul_rn(t_fix, s0);
  int mprime = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if (8 * q + j < c && sc[q] >= thr) ++mprime;
#pragma unroll
  for (int s = 1; s < 8; s <<= 1) mprime += __shfl_xor_sync(0xffffffffu, mprime, s);
  if (!write) return;
  const bool top_k_branch = (Mk >= eps_high);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int r = 8 * q + j;
    if (r < c) {
      cand_ids[r] = (uint8_t)ki[q];
      cand_scores[r] = sc[q];
    }
  }
  if (j == 0) *cstar = top_k_branch ? (uint16_t)0 : (uint16_t)max(k, mprime);
  if (fm && (top_k_branch || mprime <= k)) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (8 * q + j < k) atomicOr(&fm[ki[q]], bit);
  }
}

// One warp contracts ROWS = MT*16 consecutive tokens [tok0, tok0 + ROWS) of one layer with W_g
// and leaves their fp32 logits (+ bias) in its shared-memory tile.
// NT: 8-expert column tiles (E padded up to NT*8).  MT: 16-row tiles per warp.
// KU: chunks of 32 hidden elements issued per loop trip.
// tile: this warp's shared-memory scratch of ROWS * (NT*8 + 1) floats.
template <int NT, int MT, int KU>
__device__ __forceinline__ void router_warp(const RouteArgs& A, int layer, long long tok0,
                                            float* tile, int lane) {
  constexpr int ROWS = MT * 16;
  constexpr int EP = NT * 8;
  constexpr int LDS = EP + 1;
  const int g = lane >> 2, q = lane & 3;
  const int T = A.T, d = A.d, E = A.E;

  const uint16_t* hid = A.hidden + (size_t)(A.layer0 + layer) * A.hidden_ls;
  const uint16_t* wg = A.wg + (size_t)(A.layer0 + layer) * A.wg_ls;

  const uint16_t* arow[MT][2];
#pragma unroll
  for (int m = 0; m < MT; ++m) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      long long r = tok0 + m * 16 + h * 8 + g;
      if (r > T - 1) r = T - 1;  // rows past the end re-read the last row; results dropped
      arow[m][h] = hid + r * A.ld_h + q * 8;
    }
  }
  const uint16_t* brow[NT];
  bool bval[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int e = n * 8 + g;
    bval[n] = e < E;
    brow[n] = wg + (long long)(bval[n] ? e : 0) * A.ld_w + q * 8;
  }

  float acc[MT][NT][4];
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[m][n][i] = 0.0f;

  const int full_chunks = d / 32;
  int kc = 0;
  for (; kc + KU <= full_chunks; kc += KU) {
    uint4 av[KU][MT][2];
#pragma unroll
    for (int u = 0; u < KU; ++u)
#pragma unroll
      for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h) av[u][m][h] = ldg_stream(arow[m][h] + (kc + u) * 32);
#pragma unroll
    for (int u = 0; u < KU; ++u) {
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        uint4 b = make_uint4(0, 0, 0, 0);
        if (bval[n]) b = __ldg(reinterpret_cast<const uint4*>(brow[n] + (kc + u) * 32));
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          mma_bf16_16816(acc[m][n], av[u][m][0].x, av[u][m][1].x, av[u][m][0].y, av[u][m][1].y,
                         b.x, b.y);
          mma_bf16_16816(acc[m][n], av[u][m][0].z, av[u][m][1].z, av[u][m][0].w, av[u][m][1].w,
                         b.z, b.w);
        }
      }
    }
  }
  // remaining chunks, the last possibly partial (d is a multiple of 8)
  for (; kc * 32 < d; ++kc) {
    const bool in = (kc * 32 + q * 8 + 8) <= d;
    uint4 av[MT][2];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
      for (int h = 0; h < 2; ++h)
        av[m][h] = in ? ldg_stream(arow[m][h] + kc * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      uint4 b = make_uint4(0, 0, 0, 0);
      if (bval[n] && in) b = __ldg(reinterpret_cast<const uint4*>(brow[n] + kc * 32));
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        mma_bf16_16816(acc[m][n], av[m][0].x, av[m][1].x, av[m][0].y, av[m][1].y, b.x, b.y);
        mma_bf16_16816(acc[m][n], av[m][0].z, av[m][1].z, av[m][0].w, av[m][1].w, b.z, b.w);
      }
    }
  }

  // accumulators (+ bias) -> this warp's shared-memory tile [ROWS][LDS]
  const float* bias = A.bias ? A.bias + (size_t)(A.layer0 + layer) * E : nullptr;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int e0 = n * 8 + q * 2;
    const float b0 = (bias && e0 < E) ? bias[e0] : 0.0f;
    const float b1 = (bias && e0 + 1 < E) ? bias[e0 + 1] : 0.0f;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      float v0 = acc[m][n][0], v1 = acc[m][n][1], v2 = acc[m][n][2], v3 = acc[m][n][3];
      if (bias) {
        v0 = __fadd_rn(v0, b0); v1 = __fadd_rn(v1, b1);
        v2 = __fadd_rn(v2, b0); v3 = __fadd_rn(v3, b1);
      }
      const float big = 3.402823466e+38f;  // non-finite logits are clamped into range
      v0 = fminf(fmaxf(v0, -big), big); v1 = fminf(fmaxf(v1, -big), big);
      v2 = fminf(fmaxf(v2, -big), big); v3 = fminf(fmaxf(v3, -big), big);
      tile[(m * 16 + g) * LDS + e0] = v0;
      tile[(m * 16 + g) * LDS + e0 + 1] = v1;
      tile[(m * 16 + g + 8) * LDS + e0] = v2;
      tile[(m * 16 + g + 8) * LDS + e0 + 1] = v3;
    }
  }
  __syncwarp();

  const int rows_here = (int)min((long long)ROWS, (long long)T - tok0);
  if (A.logits_out) {
    float* out = A.logits_out + ((size_t)(A.layer0 + layer) * T + tok0) * E;
    for (int idx = lane; idx < rows_here * E; idx += 32) {
      const int r = idx / E, e = idx - r * E;
      out[idx] = tile[r * LDS + e];
    }
  }

}

// Writes the masks of one group of 32 tokens (fm, shared memory, [E]) to the workspace; called by
// a full warp after its lanes have set their bits.
__device__ __forceinline__ void publish_group_masks(const RouteArgs& A, int abs_layer, long long tok0,
                                                    const uint32_t* fm, int lane) {
  __syncwarp();
  uint32_t* out = reinterpret_cast<uint32_t*>(A.ws + (size_t)abs_layer * A.ws_ls + A.lay.fmask) +
                  (size_t)(tok0 >> 5) * A.E;
  for (int e = lane; e < A.E; e += 32) out[e] = fm[e];
}

// Score epilogue of up to 32 tokens [tok0, tok0 + 32) by one warp, lane = token; every lane of
// the warp must call.  rows: the tokens' logits in shared memory, row stride lds floats.
// fm: the warp's mask scratch in shared memory ([E] words; only used, and only needed, when
// E > 32).
__device__ __forceinline__ void group_epilogue(const RouteArgs& A, int layer, long long tok0,
                                               const float* rows, int lds, int lane,
                                               uint32_t* fm) {
  const bool masks = A.E > 32;
  if (masks) {
    for (int e = lane; e < A.E; e += 32) fm[e] = 0;
    __syncwarp();
  } else {
    fm = nullptr;
  }
  const long long t = tok0 + lane;
  if (t < A.T) {
    unsigned char* ws = A.ws + (size_t)(A.layer0 + layer) * A.ws_ls;
    const int k = A.k, c = A.c;
    uint16_t* cs_p = reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + t;
    uint8_t* ids_p = ws + A.lay.cand_ids + (size_t)t * c;
    float* sc_p = reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)t * c;
    if (A.trim_random)
      token_epilogue_random(rows + lane * lds, A.E, k, c, A.eps_high[layer], A.t_fix[layer],
                            A.renorm, A.seed, A.layer0 + layer, t, cs_p, ids_p, sc_p, fm,
                            1u << lane);
    else
      token_epilogue(rows + lane * lds, A.E, k, c, A.eps_high[layer], A.t_fix[layer], A.renorm,
                     cs_p, ids_p, sc_p, fm, 1u << lane);
  }
  if (masks) publish_group_masks(A, A.layer0 + layer, tok0, fm, lane);
}


// Router for calls with few tokens: one block routes 16 tokens, its 8 warps each contract one
// eighth of the hidden dimension (so that many SMs share the streaming of a small input),
// the partial sums meet in shared memory in a fixed order, and warps 0..3 score 4 tokens each.
// NT: 8-expert column tiles.  smem: router_splitk_smem_bytes(NT).
__host__ __device__ inline size_t router_splitk_smem_bytes(int NT) {
  return sizeof(float) * (8 * 16 * NT * 8 + 16 * (NT * 8 + 8)) + sizeof(uint32_t) * NT * 8;
}

template <int NT, int KU>
__device__ __forceinline__ void router_splitk_block(const RouteArgs& A, int layer, int rt,
                                                    float* smem) {
  constexpr int EP = NT * 8;
  constexpr int LDS = EP + 8;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, q = lane & 3;
  const int T = A.T, d = A.d, E = A.E;
  const long long tok0 = (long long)rt * 16;
  const int abs_layer = A.layer0 + layer;
  const uint16_t* hid = A.hidden + (size_t)abs_layer * A.hidden_ls;
  const uint16_t* wg = A.wg + (size_t)abs_layer * A.wg_ls;

  const uint16_t* arow[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    long long r = tok0 + h * 8 + g;
    if (r > T - 1) r = T - 1;  // rows past the end re-read the last row; results dropped
    arow[h] = hid + r * A.ld_h + q * 8;
  }
  const uint16_t* brow[NT];
  bool bval[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int e = n * 8 + g;
    bval[n] = e < E;
    brow[n] = wg + (long long)(bval[n] ? e : 0) * A.ld_w + q * 8;
  }
  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[n][i] = 0.0f;

  // this warp's chunks of 32 hidden elements: [c_begin, c_end)
  const int chunks = (d + 31) / 32;
  const int per = (chunks + 7) / 8;
  const int c_begin = min(chunks, warp * per), c_end = min(chunks, c_begin + per);
  int kc = c_begin;
  // all fragments of KU chunks are requested before the first MMA: with 16 tokens per block
  // there are few warps per SM, so the loads of one warp must overlap each other
  for (; kc + KU <= c_end && (kc + KU) * 32 <= d; kc += KU) {
    uint4 av[KU][2];
    uint4 bv[KU][NT];
#pragma unroll
    for (int u = 0; u < KU; ++u) {
#pragma unroll
      for (int h = 0; h < 2; ++h) av[u][h] = ldg_stream(arow[h] + (kc + u) * 32);
#pragma unroll
      for (int n = 0; n < NT; ++n)
        bv[u][n] = bval[n] ? __ldg(reinterpret_cast<const uint4*>(brow[n] + (kc + u) * 32))
                           : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < KU; ++u) {
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        mma_bf16_16816(acc[n], av[u][0].x, av[u][1].x, av[u][0].y, av[u][1].y, bv[u][n].x,
                       bv[u][n].y);
        mma_bf16_16816(acc[n], av[u][0].z, av[u][1].z, av[u][0].w, av[u][1].w, bv[u][n].z,
                       bv[u][n].w);
      }
    }
  }
  for (; kc < c_end; ++kc) {   // remaining chunks, the last possibly partial
    const bool in = (kc * 32 + q * 8 + 8) <= d;
    uint4 av[2];
#pragma unroll
    for (int h = 0; h < 2; ++h)
      av[h] = in ? ldg_stream(arow[h] + kc * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      uint4 b = make_uint4(0, 0, 0, 0);
      if (bval[n] && in) b = __ldg(reinterpret_cast<const uint4*>(brow[n] + kc * 32));
      mma_bf16_16816(acc[n], av[0].x, av[1].x, av[0].y, av[1].y, b.x, b.y);
      mma_bf16_16816(acc[n], av[0].z, av[1].z, av[0].w, av[1].w, b.z, b.w);
    }
  }

  // partial sums -> shared memory [warp][16][EP]
  float* part = smem + (size_t)warp * 16 * EP;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int e0 = n * 8 + q * 2;
    part[g * EP + e0] = acc[n][0];
    part[g * EP + e0 + 1] = acc[n][1];
    part[(g + 8) * EP + e0] = acc[n][2];
    part[(g + 8) * EP + e0 + 1] = acc[n][3];
  }
  __syncthreads();
  // logits = ((p0 + p1) + ... + p7) + bias, clamped; tile rows are LDS floats apart
  float* tile = smem + 8 * 16 * EP;
  // masks of the tile's tokens without a load-dependent choice (16 tokens: half a group)
  uint32_t* fm = E > 32 ? reinterpret_cast<uint32_t*>(tile + 16 * LDS) : nullptr;
  if (fm)
    for (int e = tid; e < E; e += blockDim.x) fm[e] = 0;
  const float* bias = A.bias ? A.bias + (size_t)abs_layer * E : nullptr;
  const float big = 3.402823466e+38f;
  for (int idx = tid; idx < 16 * EP; idx += blockDim.x) {
    const int r = idx / EP, e = idx - r * EP;
    float v = smem[idx];
#pragma unroll
    for (int w = 1; w < 8; ++w) v = __fadd_rn(v, smem[w * 16 * EP + idx]);
    if (bias && e < E) v = __fadd_rn(v, bias[e]);
    tile[r * LDS + e] = fminf(fmaxf(v, -big), big);
  }
  __syncthreads();
  const int rows_here = (int)min(16LL, (long long)T - tok0);
  if (A.logits_out) {
    float* out = A.logits_out + ((size_t)abs_layer * T + tok0) * E;
    for (int idx = tid; idx < rows_here * E; idx += blockDim.x) {
      const int r = idx / E, e = idx - r * E;
      out[idx] = tile[r * LDS + e];
    }
  }
  if (A.trim_random) {
    const long long t = tok0 + tid;
    if (tid < 16 && t < T) {
      unsigned char* ws = A.ws + (size_t)abs_layer * A.ws_ls;
      const int k = A.k, c = A.c;
      token_epilogue_random(tile + (size_t)tid * LDS, E, k, c, A.eps_high[layer], A.t_fix[layer],
                            A.renorm, A.seed, abs_layer, t,
                            reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + t,
                            ws + A.lay.cand_ids + (size_t)t * c,
                            reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)t * c,
                            fm, 1u << tid);
    }
  } else if (warp < 4) {
    const int r = warp * 4 + (lane >> 3);
    const long long t = tok0 + r;
    const bool write = t < T;
    const long long tc = write ? t : 0;
    unsigned char* ws = A.ws + (size_t)abs_layer * A.ws_ls;
    const int k = A.k, c = A.c;
    token_epilogue_lanes8<EP>(tile + (size_t)r * LDS, lane & 7, E, k, c, A.eps_high[layer],
                              A.t_fix[layer], A.renorm, write,
                              reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + tc,
                              ws + A.lay.cand_ids + (size_t)tc * c,
                              reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)tc * c,
                              fm, 1u << r);
  }
  if (fm) {
    __syncthreads();
    // this tile's 16-bit half of the group's mask words
    uint16_t* out = reinterpret_cast<uint16_t*>(A.ws + (size_t)abs_layer * A.ws_ls + A.lay.fmask) +
                    ((size_t)(rt >> 1) * E) * 2 + (rt & 1);
    for (int e = tid; e < E; e += blockDim.x) out[2 * e] = (uint16_t)fm[e];
    if ((rt & 1) == 0 && tok0 + 16 >= T)   // the group's upper half has no tokens: zero it
      for (int e = tid; e < E; e += blockDim.x) out[2 * e + 1] = 0;
  }
}

}  // namespace laser
