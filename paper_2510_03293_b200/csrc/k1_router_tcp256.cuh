// Scoring team of the persistent tensor-memory router for 128 < E <= 256 and c <= 16: one thread
// per token reads its 256 accumulator columns straight from tensor memory, 32 at a time, in
// three passes (there is no room for a logits tile next to four 48 KB stages):
//   pass A  x = accumulator + bias, clamped; the row maximum; the logits output if asked for
//   pass B  e = exp32(x - max) into the eight interleaved sums; every x becomes a 32-bit key
//           (order-preserving bits of x, low 8 bits replaced by 255 - index); groups of 16 keys
//           are sorted by a bitonic network and merged into the 16 best so far
//   pass C  the exact x of the 16 listed experts (each chunk passes through the thread's
//           scratch row so that it can be indexed)
// The accumulator is handed back after pass C.  Dropping the low bits of x can misplace only
// logits that agree in all kept bits.  If the kept bits of the c-th listed key exceed those of
// the best key outside the list, the c best experts by (x descending, index ascending) are in
// the list, and ordering the list by its exact values gives their ranks; otherwise the token
// is redone from a full row by token_epilogue (the warp reads the row again, one such token at
// a time).  The softmax is that of token_epilogue, operation by operation.
#pragma once
#include "k1_router_tc.cuh"

namespace laser {

constexpr int kTcp256Scratch = 32 * 33;   // floats per warp: one padded 32-float row per lane

// x of one accumulator chunk: + bias, clamped into the finite range
__device__ __forceinline__ void tcp256_chunk(uint32_t taddr, const float* bias_c, bool has_bias,
                                             float (&x)[32]) {
  const float big = 3.402823466e+38f;
  tc_ld32(taddr, x);
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const float xv = has_bias ? __fadd_rn(x[i], bias_c[i]) : x[i];
    x[i] = fminf(fmaxf(xv, -big), big);
  }
}

// The team (warps 0..3) of a persistent router block with 256 accumulator columns.
// scratch: 4 * kTcp256Scratch floats; the other arguments as for router_tcp_team.
__device__ __forceinline__ void router_tcp256_team(const RouteArgs& A, int n_layers, int first,
                                                   int step, int n_tiles, uint32_t tmem,
                                                   float* scratch, float* bias_s, uint32_t* s_fm,
                                                   uint64_t* acc_full, uint64_t* acc_empty,
                                                   volatile int* abort) {
  constexpr int N = 256, CL = 16;
  constexpr uint32_t IDX = N - 1;
  constexpr int SH = 8;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = A.T, E = A.E, k = A.k, c = A.c;
  const bool has_bias = A.bias != nullptr;
  float* wscr = scratch + warp * kTcp256Scratch;   // the warp's scratch
  float* myrow = wscr + lane * 33;                 // this thread's 32-float row
  uint32_t* fm = s_fm + warp * N;                  // masks of this warp's group of 32 tokens
  int j = 0;
  for (int tile_id = first; tile_id < n_tiles; tile_id += step, ++j) {
    const int layer = tile_id % n_layers, rt = tile_id / n_layers, a = j & 1;
    const int abs_layer = A.layer0 + layer;
    for (int e = tid; e < N; e += 128)
      bias_s[e] = (has_bias && e < E) ? A.bias[(size_t)abs_layer * E + e] : 0.0f;
    for (int e = lane; e < N; e += 32) fm[e] = 0;
    bool ok = true;
    if (lane == 0) ok = tc_mbar_wait(acc_full + a, (uint32_t)((j >> 1) & 1), abort);
    if (!__shfl_sync(0xffffffffu, ok ? 1 : 0, 0) && lane == 0 && !*abort) {
      *abort = 1;
      if (A.status) atomicOr(A.status, 2);
    }
    team_barrier();   // the bias is in place; every warp has seen its accumulator (or given up)
    int* ready = reinterpret_cast<int*>(A.ws + (size_t)abs_layer * A.ws_ls + A.lay.ready);
    if (*abort) {
      if (tid == 0 && rt != A.withhold_tile) { __threadfence(); st_release(ready + rt, -1); }
      break;
    }
    tc_fence_after();
    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(a * N);
    const long long tok0 = (long long)rt * kTcTileM;
    const long long t = tok0 + tid;
    const bool live = t < T;
    const float eps_high = A.eps_high[layer], t_fix = A.t_fix[layer];
    unsigned char* ws = A.ws + (size_t)abs_layer * A.ws_ls;
    uint16_t* cs_p = reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + (live ? t : 0);
    uint8_t* ids_p = ws + A.lay.cand_ids + (size_t)(live ? t : 0) * c;
    float* sc_p = reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)(live ? t : 0) * c;

    // ---- pass A: maximum (and the logits, if the caller wants them)
    float xmax;
    {
      float m[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) m[q] = __int_as_float(0xff800000);
      float* out = (A.logits_out && live) ? A.logits_out + ((size_t)abs_layer * T + t) * E : nullptr;
#pragma unroll 1
      for (int ch = 0; ch < N / 32; ++ch) {
        float x[32];
        tcp256_chunk(taddr + ch * 32, bias_s + ch * 32, has_bias, x);
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (ch * 32 + i < E) m[i & 3] = fmaxf(m[i & 3], x[i]);
        if (out) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (ch * 32 + i < E) out[ch * 32 + i] = x[i];
        }
      }
      xmax = fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
    }

    // ---- pass B: the softmax denominator and the 16 best keys
    float sum8[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) sum8[q] = 0.0f;
    uint32_t R[CL];   // the CL best keys so far, descending
    uint32_t dm = 0;  // the best key that is not in R
#pragma unroll
    for (int i = 0; i < CL; ++i) R[i] = 0;
#pragma unroll 1
    for (int ch = 0; ch < N / 32; ++ch) {
      float x[32];
      tcp256_chunk(taddr + ch * 32, bias_s + ch * 32, has_bias, x);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t B[CL];
        float ev[CL];
#pragma unroll
        for (int i = 0; i < CL; ++i) ev[i] = exp32(__fsub_rn(x[h * CL + i], xmax));
#pragma unroll
        for (int i = 0; i < CL; ++i) {
          const int e = ch * 32 + h * CL + i;
          const bool in = e < E;
          // CL is a multiple of 8: element e adds to sum e mod 8, in ascending order of e
          sum8[i & 7] = __fadd_rn(sum8[i & 7], in ? ev[i] : 0.0f);
          const uint32_t u = __float_as_uint(x[h * CL + i]);
          const uint32_t o = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
          B[i] = in ? ((o & ~IDX) | (IDX - (uint32_t)e)) : 0u;
        }
        sort_desc<CL>(B);
        if (ch == 0 && h == 0) {
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
    }
    const float Z = __fadd_rn(__fadd_rn(__fadd_rn(sum8[0], sum8[1]), __fadd_rn(sum8[2], sum8[3])),
                              __fadd_rn(__fadd_rn(sum8[4], sum8[5]), __fadd_rn(sum8[6], sum8[7])));
    uint32_t rc = 0;   // the c-th listed key
#pragma unroll
    for (int i = 0; i < CL; ++i)
      if (i == c - 1) rc = R[i];
    const bool exact = (rc >> SH) > (dm >> SH);

    // ---- pass C: the exact logits of the listed experts
    float xl[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) xl[r] = 0.0f;
#pragma unroll 1
    for (int ch = 0; ch < N / 32; ++ch) {
      float x[32];
      tcp256_chunk(taddr + ch * 32, bias_s + ch * 32, has_bias, x);
#pragma unroll
      for (int i = 0; i < 32; ++i) myrow[i] = x[i];
#pragma unroll
      for (int r = 0; r < CL; ++r) {
        const uint32_t e = IDX - (R[r] & IDX);
        if ((int)(e >> 5) == ch) xl[r] = myrow[e & 31];
      }
    }

    // ---- tokens whose list may miss one of the c best: redone from the full row, one at a time
    uint32_t redo = __ballot_sync(0xffffffffu, live && !exact);
    while (redo) {
      const int src = __ffs(redo) - 1;
      redo &= redo - 1;
      __syncwarp();
#pragma unroll 1
      for (int ch = 0; ch < N / 32; ++ch) {
        float x[32];
        tcp256_chunk(taddr + ch * 32, bias_s + ch * 32, has_bias, x);
        if (lane == src) {
#pragma unroll
          for (int i = 0; i < 32; ++i) wscr[ch * 32 + i] = x[i];
        }
      }
      if (lane == src)
        token_epilogue(wscr, E, k, c, eps_high, t_fix, A.renorm, cs_p, ids_p, sc_p, fm, 1u << lane);
      __syncwarp();
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) tcp_mbar_arrive(acc_empty + a);   // the issuer may reuse the accumulator

    if (live && exact) {
      // order the list by (x descending, index ascending): the key order already is that order
      // except inside runs of equal kept bits
      uint32_t id[CL], ko[CL];
#pragma unroll
      for (int r = 0; r < CL; ++r) {
        id[r] = IDX - (R[r] & IDX);
        const uint32_t u = __float_as_uint(xl[r]);
        ko[r] = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
      }
      bool swapped;
      do {
        swapped = false;
#pragma unroll
        for (int r = 0; r + 1 < CL; ++r) {
          const bool sw = ko[r] < ko[r + 1] || (ko[r] == ko[r + 1] && id[r] > id[r + 1]);
          const uint32_t k0 = ko[r], k1 = ko[r + 1], i0 = id[r], i1 = id[r + 1];
          const float x0 = xl[r], x1 = xl[r + 1];
          ko[r] = sw ? k1 : k0; ko[r + 1] = sw ? k0 : k1;
          id[r] = sw ? i1 : i0; id[r + 1] = sw ? i0 : i1;
          xl[r] = sw ? x1 : x0; xl[r + 1] = sw ? x0 : x1;
          swapped = swapped || sw;
        }
      } while (swapped);
      float sv[CL];
#pragma unroll
      for (int r = 0; r < CL; ++r) sv[r] = __fdiv_rn(exp32(__fsub_rn(xl[r], xmax)), Z);
      float Mk = 0.0f, thr = 0.0f;
      int mprime = 0;
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
      *cs_p = top_k_branch ? (uint16_t)0 : (uint16_t)max(k, mprime);
      if (top_k_branch || mprime <= k) {
#pragma unroll
        for (int r = 0; r < CL; ++r)
          if (r < k) atomicOr(&fm[id[r]], 1u << lane);
      }
      if (c == CL) {   // 16 ids = 16 bytes, 16 scores = 64 bytes, both aligned for this c
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          w[q] = id[4 * q] | (id[4 * q + 1] << 8) | (id[4 * q + 2] << 16) | (id[4 * q + 3] << 24);
        *reinterpret_cast<uint4*>(ids_p) = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<float4*>(sc_p + 4 * q) =
              make_float4(sv[4 * q], sv[4 * q + 1], sv[4 * q + 2], sv[4 * q + 3]);
      } else {
#pragma unroll
        for (int r = 0; r < CL; ++r) {
          if (r < c) { ids_p[r] = (uint8_t)id[r]; sc_p[r] = sv[r]; }
        }
      }
    }
    if (tok0 + warp * 32 < T) publish_group_masks(A, abs_layer, tok0 + warp * 32, fm, lane);
    team_barrier();   // every record of the tile is written
    if (tid == 0 && rt != A.withhold_tile) { __threadfence(); st_release(ready + rt, 1); }
  }
}

}  // namespace laser
