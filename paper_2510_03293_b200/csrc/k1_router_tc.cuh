// K1 for E > 32: the router contraction x = h.W_g^T + b on the 5th-generation tensor cores
// (tcgen05.mma, accumulator in tensor memory) with operands brought in by TMA, fused with the
// per-token score epilogue.
//
// One thread block routes one tile of 128 tokens of one layer:
//   warp 0, one lane   producer: per 64-element slice of the hidden dimension one TMA load of
//                      the 128 x 64 hidden tile and one of the N x 64 W_g tile (128-byte
//                      swizzle) into a ring of shared-memory stages, completion on mbarriers
//   warp 1, one lane   issues four m128 x nN x k16 bf16 MMAs per stage into N fp32 columns of
//                      tensor memory; tcgen05.commit releases the stage / publishes the tile
//   all 8 warps        epilogue, once the accumulator is complete: the logits (+ bias) go from
//                      tensor memory through registers into the now idle stage memory; then
//                      N <= 128: warps 0..3 score one token per thread, ranking the experts
//                      with sorting networks on 32-bit keys (token_epilogue_sorted);
//                      N = 256: groups of 8 lanes score one token each (lane j owns the
//                      experts i = j mod 8; every reduction is a 3-step butterfly).
// Rows past the end of a layer and expert columns >= E hold other rows' data or zeros; they
// are computed and ignored.  Every wait is bounded; a wait that runs out raises the timeout
// bit, and the block still drains its copies and frees its tensor memory before it returns.
#pragma once
#include <cuda.h>

#include "k1_router.cuh"
#include "k2_select.cuh"

namespace laser {

constexpr int kTcTileM = 128;       // tokens per tile (MMA M)
constexpr int kTcSliceK = 64;       // bf16 elements per stage row = 128 bytes = one swizzle row
constexpr long long kTcWaitCycles = 2000000000LL;   // give up a wait after ~1 s

template <int N>
__host__ __device__ constexpr int tc_stage_bytes() { return (kTcTileM + N) * kTcSliceK * 2; }
// N = 64 keeps two stages (48 KB) so that four blocks fit one SM and their streaming and scoring
// phases overlap; the wider shapes need the stage memory for the logits tile of the epilogue.
template <int N>
__host__ __device__ constexpr int tc_stages() {
  return N <= 64 ? 2 : (96 * 1024) / tc_stage_bytes<N>();
}
template <int N>
__host__ __device__ constexpr int tc_min_blocks() { return N <= 64 ? 4 : 2; }
// stages (1024-byte aligned, hence the slack) + bias + barriers
template <int N>
__host__ __device__ constexpr size_t tc_smem_bytes() {
  return 1024 + (size_t)tc_stages<N>() * tc_stage_bytes<N>() + sizeof(float) * N + 256;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void tc_mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count)
               : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes) : "memory");
}
__device__ __forceinline__ bool tc_mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait; gives up at once when *abort is raised by another role of the block.
__device__ __forceinline__ bool tc_mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  if (tc_mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  while (!tc_mbar_try_wait(bar, parity)) {
    if (*abort || clock64() - start > kTcWaitCycles) return false;
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar,
                                            int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)),
        "r"(c0), "r"(c1) : "memory");
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes (64 bf16) stored
// with the 128-byte swizzle; groups of 8 rows are 1024 bytes apart.
//   bits 0-13  start address >> 4        bits 16-29  leading offset (1: unused when swizzled)
//   bits 32-45 stride between 8-row groups >> 4
//   bits 46-47 descriptor version 1      bits 61-63  layout 2 = 128-byte swizzle
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) |
         ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, both K-major.
//   bits 4-5 D format (1 = f32), 7-9 A format (1 = bf16), 10-12 B format (1 = bf16),
//   bits 17-22 N >> 3, bits 24-28 M >> 4
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                       uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Router role of one block (256 threads) for tile `rt` (128 tokens) of local layer `layer`.
// N: accumulator columns, a multiple of 16 with E <= N <= 256.
// Returns false if one of the block's own waits ran out (no records were written then).
template <int N, int CL>
__device__ __forceinline__ bool router_tc_block(const RouteArgs& A, const CUtensorMap* map_h,
                                                const CUtensorMap* map_w, int layer, int rt,
                                                unsigned char* dyn_smem) {
  constexpr int STAGES = tc_stages<N>();
  constexpr int STAGE_BYTES = tc_stage_bytes<N>();
  constexpr int A_BYTES = kTcTileM * kTcSliceK * 2;
  constexpr int TMEM_COLS = N <= 32 ? 32 : (N <= 64 ? 64 : (N <= 128 ? 128 : 256));
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ uint32_t s_fm[4 * N];   // masks of the tile's four groups (see group_epilogue)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = A.T, E = A.E, d = A.d;
  const int abs_layer = A.layer0 + layer;

  unsigned char* stages =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~uintptr_t(1023));
  float* bias_s = reinterpret_cast<float*>(stages + (size_t)STAGES * STAGE_BYTES);
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + N);   // [STAGES] TMA landed
  uint64_t* empty = full + STAGES;                            // [STAGES] MMAs of the stage done
  uint64_t* acc_bar = empty + STAGES;                         // accumulator complete

  // Tensor memory first: the SM starts the next block of this kernel only after this one has
  // given up its right to allocate (measured: blocks of an SM start 1.2 us apart).
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&s_tmem)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const int nk = (d + kTcSliceK - 1) / kTcSliceK;
  // rows of the [layers*T, d] and [layers*E, d] views (the launcher keeps both below 2^31)
  const int row_h = abs_layer * T + rt * kTcTileM;
  const int row_w = abs_layer * E;
  const int first_fill = nk < STAGES ? nk : STAGES;   // stage fills that need no free stage

  const bool has_bias = A.bias != nullptr;
  if (tid == 0) {
    // the producer thread: barriers, then the first loads at once, before the block meets
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) { tc_mbar_init(full + s, 1); tc_mbar_init(empty + s, 1); }
    tc_mbar_init(acc_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int kc = 0; kc < first_fill; ++kc) {
      unsigned char* sa = stages + (size_t)kc * STAGE_BYTES;
      tc_mbar_expect_tx(full + kc, (uint32_t)STAGE_BYTES);
      tma_load_2d(sa, map_h, full + kc, kc * kTcSliceK, row_h);
      tma_load_2d(sa + A_BYTES, map_w, full + kc, kc * kTcSliceK, row_w);
    }
  }
  for (int e = tid; e < N; e += blockDim.x)
    bias_s[e] = (has_bias && e < E) ? A.bias[(size_t)abs_layer * E + e] : 0.0f;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abort = &s_abort;

  if (warp == 0 && lane == 0) {
    // producer
    int issued = first_fill;
    for (int kc = first_fill; kc < nk; ++kc) {
      const int s = kc % STAGES, use = kc / STAGES;
      if (use > 0 && !tc_mbar_wait(empty + s, (uint32_t)((use - 1) & 1), abort)) break;
      unsigned char* sa = stages + (size_t)s * STAGE_BYTES;
      tc_mbar_expect_tx(full + s, (uint32_t)STAGE_BYTES);
      tma_load_2d(sa, map_h, full + s, kc * kTcSliceK, row_h);
      tma_load_2d(sa + A_BYTES, map_w, full + s, kc * kTcSliceK, row_w);
      issued = kc + 1;
    }
    if (issued < nk) {
      // gave up: make the others stop, then let the copies already issued land
      if (!*abort) { *abort = 1; if (A.status) atomicOr(A.status, 2); }
      for (int kc = max(0, issued - STAGES); kc < issued; ++kc) {
        const long long start = clock64();
        while (!tc_mbar_try_wait(full + kc % STAGES, (uint32_t)((kc / STAGES) & 1)))
          if (clock64() - start > kTcWaitCycles) break;
      }
    }
  } else if (warp == 1 && lane == 0) {
    // MMA issuer
    constexpr uint32_t idesc = tc_idesc(kTcTileM, N);
    bool ok = true;
    for (int kc = 0; kc < nk && ok; ++kc) {
      const int s = kc % STAGES, use = kc / STAGES;
      if (!tc_mbar_wait(full + s, (uint32_t)(use & 1), abort)) { ok = false; break; }
      tc_fence_after();
      const uint32_t sa = smem_u32(stages + (size_t)s * STAGE_BYTES);
      const uint64_t adesc = tc_smem_desc(sa), bdesc = tc_smem_desc(sa + A_BYTES);
#pragma unroll
      for (int kk = 0; kk < kTcSliceK / 16; ++kk)   // 16 elements = 32 bytes = 2 address units
        tc_mma(tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kc > 0 || kk > 0) ? 1u : 0u);
      tc_commit(empty + s);
    }
    if (ok) tc_commit(acc_bar);
    else if (!*abort) { *abort = 1; if (A.status) atomicOr(A.status, 2); }
  }
  __syncwarp();

  // ---- epilogue, all 8 warps ------------------------------------------------------------
  // One lane polls for the accumulator; everybody else sleeps in the block barrier, so that the
  // issue slots of the SM go to the blocks that are scoring or issuing copies.
  bool acc_ok = true;
  if (warp == 2 && lane == 0) acc_ok = tc_mbar_wait(acc_bar, 0u, abort);
  const bool gave_up = __syncthreads_or(acc_ok ? 0 : 1) != 0;
  if (gave_up) {
    if (tid == 0 && A.status) atomicOr(A.status, 2);
  } else {
    tc_fence_after();
    // Every stage has been read by its MMAs, so the stage memory now holds the logits tile.
    const float big = 3.402823466e+38f;  // non-finite logits are clamped into range
    const int k = A.k, c = A.c;
    unsigned char* ws = A.ws + (size_t)abs_layer * A.ws_ls;
    float* tile = reinterpret_cast<float*>(stages);
    for (int i = tid; i < 4 * N; i += blockDim.x) s_fm[i] = 0;   // (a block barrier follows)
    if constexpr (N <= 128) {
      // N <= 128: all 128 rows of N + 1 floats (odd stride: a thread per row is conflict-free),
      // then warps 0..3 score one token per thread with sorting networks
      constexpr int LDS = N + 1;
      static_assert(128 * LDS * 4 <= STAGES * STAGE_BYTES, "tile must fit the stage memory");
      {
        // tensor memory -> registers -> shared memory: warp w reads TMEM lanes 32*(w%4)..+31
        // (its quadrant) and the column half w/4
        const int q = warp & 3, h = warp >> 2;
        float* dst = tile + (size_t)(q * 32 + lane) * LDS;
        float v[32];
#pragma unroll 1
        for (int ch = h * (N / 64); ch < (h + 1) * (N / 64); ++ch) {
          tc_ld32(tmem + ((uint32_t)(q * 32) << 16) + ch * 32, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int e = ch * 32 + i;
            float xv = has_bias ? __fadd_rn(v[i], bias_s[e]) : v[i];
            dst[e] = fminf(fmaxf(xv, -big), big);
          }
        }
      }
      __syncthreads();
      const long long tok0 = (long long)rt * kTcTileM;
      if (A.logits_out) {
        const int rows_here = (int)max(0LL, min(128LL, (long long)T - tok0));
        float* out = A.logits_out + ((size_t)abs_layer * T + tok0) * E;
        for (int idx = tid; idx < rows_here * E; idx += blockDim.x) {
          const int r = idx / E, e = idx - r * E;
          out[idx] = tile[r * LDS + e];
        }
      }
      const long long t = tok0 + tid;
      uint32_t* fm = s_fm + warp * N;   // warps 0..3 each score one group of 32 tokens
      if (tid < kTcTileM && t < T) {
        uint16_t* cs_p = reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + t;
        uint8_t* ids_p = ws + A.lay.cand_ids + (size_t)t * c;
        float* sc_p = reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)t * c;
        if (A.trim_random)
          token_epilogue_random(tile + (size_t)tid * LDS, E, k, c, A.eps_high[layer],
                                A.t_fix[layer], A.renorm, A.seed, abs_layer, t, cs_p, ids_p, sc_p,
                                fm, 1u << lane);
        else if (c <= CL)
          token_epilogue_sorted<N, CL>(tile + (size_t)tid * LDS, E, k, c, A.eps_high[layer],
                                       A.t_fix[layer], A.renorm, cs_p, ids_p, sc_p, fm,
                                       1u << lane);
        else
          token_epilogue(tile + (size_t)tid * LDS, E, k, c, A.eps_high[layer], A.t_fix[layer],
                         A.renorm, cs_p, ids_p, sc_p, fm, 1u << lane);
      }
      if (warp < 4 && tok0 + warp * 32 < T)
        publish_group_masks(A, abs_layer, tok0 + warp * 32, fm, lane);
    } else {
    // N = 256: ROWS rows of N + 8 floats (the padding keeps the four 8-lane groups of a warp on
    // different banks), the 128 tokens in two passes of 64; 8 lanes score one token.
    constexpr int LDS = N + 8;
    constexpr int ROWS = (128 * LDS * 4 <= STAGES * STAGE_BYTES) ? 128 : 64;
#pragma unroll 1
    for (int row0 = 0; row0 < kTcTileM; row0 += ROWS) {
      // tensor memory -> registers -> shared memory: warp w reads TMEM lanes 32*(w%4)..+31
      // (its quadrant) and the column half w/4
      const int q = warp & 3, h = warp >> 2;
      if (q * 32 >= row0 && q * 32 < row0 + ROWS) {
        float* dst = tile + (size_t)(q * 32 - row0 + lane) * LDS;
        float v[32];
#pragma unroll 1
        for (int ch = h * (N / 64); ch < (h + 1) * (N / 64); ++ch) {
          tc_ld32(tmem + ((uint32_t)(q * 32) << 16) + ch * 32, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int e = ch * 32 + i;
            float xv = has_bias ? __fadd_rn(v[i], bias_s[e]) : v[i];
            dst[e] = fminf(fmaxf(xv, -big), big);
          }
        }
      }
      __syncthreads();
      const long long tok0 = (long long)rt * kTcTileM + row0;
      if (A.logits_out) {
        const int rows_here = (int)max(0LL, min((long long)ROWS, (long long)T - tok0));
        float* out = A.logits_out + ((size_t)abs_layer * T + tok0) * E;
        for (int idx = tid; idx < rows_here * E; idx += blockDim.x) {
          const int r = idx / E, e = idx - r * E;
          out[idx] = tile[r * LDS + e];
        }
      }
      if (A.trim_random) {   // one thread per token of this pass
        const long long t = tok0 + tid;
        if (tid < ROWS && t < T) {
          token_epilogue_random(tile + (size_t)tid * LDS, E, k, c, A.eps_high[layer],
                                A.t_fix[layer], A.renorm, A.seed, abs_layer, t,
                                reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + t,
                                ws + A.lay.cand_ids + (size_t)t * c,
                                reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)t * c,
                                s_fm + ((row0 + tid) >> 5) * N, 1u << (tid & 31));
        }
      }
      // groups of 8 lanes score one token each, 4 tokens per warp at a time
      const int g = lane >> 3, j = lane & 7;
#pragma unroll 1
      for (int it = 0; it < (A.trim_random ? 0 : ROWS / 32); ++it) {
        const int r = warp * (ROWS / 8) + it * 4 + g;
        const long long t = tok0 + r;
        const bool write = t < T;
        const long long tc = write ? t : 0;   // keeps the pointers of idle groups in bounds
        token_epilogue_lanes8<N>(tile + (size_t)r * LDS, j, E, k, c, A.eps_high[layer],
                                 A.t_fix[layer], A.renorm, write,
                                 reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + tc,
                                 ws + A.lay.cand_ids + (size_t)tc * c,
                                 reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)tc * c,
                                 s_fm + ((row0 + r) >> 5) * N, 1u << (r & 31));
      }
      __syncthreads();   // the tile is reused by the next pass
    }
    // the masks of the tile's groups (every warp has passed the barrier above)
    if (warp < 4 && (long long)rt * kTcTileM + warp * 32 < T)
      publish_group_masks(A, abs_layer, (long long)rt * kTcTileM + warp * 32, s_fm + warp * N, lane);
  }
    }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
  return !gave_up;
}

}  // namespace laser
