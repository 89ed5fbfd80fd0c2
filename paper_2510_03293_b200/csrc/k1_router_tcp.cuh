// K1 for 32 < E <= 64 as a persistent block: the tcgen05 router of k1_router_tc.cuh with the
// three phases of a tile (streaming, contraction, scoring) running at the same time on different
// tiles, so that the block's TMA loads never pause.
//
// A router block walks the tiles b, b + P, b + 2P, ... (tile id = 128-token tile index *
// n_layers + layer, so that all layers advance together).  Roles:
//   warp 4, one lane   producer: TMA loads of the hidden and W_g slices into a ring of stages
//   warp 5, one lane   issues the MMAs of tile j into tensor-memory accumulator j % 2 and
//                      commits the stage / the accumulator
//   warps 0..3         the scoring team, one thread per token: accumulator (+ bias) from tensor
//                      memory into the thread's own row of shared memory, accumulator handed
//                      back, then the score epilogue of k1_router.cuh on that row, the group's
//                      masks, and the tile's ready flag
//   warps 6, 7         leave at once
// Every wait is bounded (the abort flag of k1_router_tc.cuh); a role that gives up raises the
// timeout bit, and the team then publishes its tile as failed (-1).
#pragma once
#include "k1_router_tc.cuh"

namespace laser {

template <int N>
__host__ __device__ constexpr int tcp_stages() { return N <= 64 ? 3 : (N == 256 ? 4 : 2); }
template <int N>
__host__ __device__ constexpr size_t tcp_tile_bytes() {
  // N = 256 scores from tensor memory and keeps only a 32-float row per thread of the team
  return N == 256 ? (size_t)4 * 32 * 33 * 4 : (size_t)kTcTileM * (N + 1) * 4;
}
// stages (1024-byte aligned, hence the slack) + logits rows + bias + barriers
template <int N>
__host__ __device__ constexpr size_t tcp_smem_bytes() {
  return 1024 + (size_t)tcp_stages<N>() * tc_stage_bytes<N>() + tcp_tile_bytes<N>() +
         sizeof(float) * N + 256;
}

__device__ __forceinline__ void tcp_mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void team_barrier() {   // the 128 threads of warps 0..3
  asm volatile("bar.sync 2, 128;" ::: "memory");
}
__device__ __forceinline__ void roles_barrier() {  // the 192 threads of warps 0..5
  asm volatile("bar.sync 3, 192;" ::: "memory");
}

// The scoring team (warps 0..3) of a persistent router block.
template <int N, int CL>
__device__ __forceinline__ void router_tcp_team(const RouteArgs& A, int n_layers, int first,
                                                int step, int n_tiles, uint32_t tmem, float* tile,
                                                float* bias_s, uint32_t* s_fm, uint64_t* acc_full,
                                                uint64_t* acc_empty, volatile int* abort) {
  constexpr int LDS = N + 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = A.T, E = A.E, k = A.k, c = A.c;
  const bool has_bias = A.bias != nullptr;
  const float big = 3.402823466e+38f;  // non-finite logits are clamped into range
  float* row = tile + (size_t)tid * LDS;       // this thread's token: a private row
  uint32_t* fm = s_fm + warp * N;              // this warp's group of 32 tokens
  int j = 0;
  for (int tile_id = first; tile_id < n_tiles; tile_id += step, ++j) {
    const int layer = tile_id % n_layers, rt = tile_id / n_layers, a = j & 1;
    const int abs_layer = A.layer0 + layer;
    if (tid < N) bias_s[tid] = (has_bias && tid < E) ? A.bias[(size_t)abs_layer * E + tid] : 0.0f;
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
      // no records for this tile: say so, which ends the layer's selection
      if (tid == 0 && rt != A.withhold_tile) { __threadfence(); st_release(ready + rt, -1); }
      break;
    }
    tc_fence_after();
    // tensor memory -> registers -> this thread's row (warp w reads its own 32 TMEM lanes)
    {
      float v[32];
#pragma unroll 1
      for (int ch = 0; ch < N / 32; ++ch) {
        tc_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(a * N + ch * 32), v);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int e = ch * 32 + i;
          const float xv = has_bias ? __fadd_rn(v[i], bias_s[e]) : v[i];
          row[e] = fminf(fmaxf(xv, -big), big);
        }
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) tcp_mbar_arrive(acc_empty + a);   // the issuer may reuse the accumulator
    const long long tok0 = (long long)rt * kTcTileM;
    const long long t = tok0 + tid;
    if (t < T) {
      unsigned char* ws = A.ws + (size_t)abs_layer * A.ws_ls;
      if (A.logits_out) {
        float* out = A.logits_out + ((size_t)abs_layer * T + t) * E;
        for (int e = 0; e < E; ++e) out[e] = row[e];
      }
      uint16_t* cs_p = reinterpret_cast<uint16_t*>(ws + A.lay.cstar) + t;
      uint8_t* ids_p = ws + A.lay.cand_ids + (size_t)t * c;
      float* sc_p = reinterpret_cast<float*>(ws + A.lay.cand_scores) + (size_t)t * c;
      if (A.trim_random)
        token_epilogue_random(row, E, k, c, A.eps_high[layer], A.t_fix[layer], A.renorm, A.seed,
                              abs_layer, t, cs_p, ids_p, sc_p, fm, 1u << lane);
      else if (c <= CL)
        token_epilogue_sorted<N, CL>(row, E, k, c, A.eps_high[layer], A.t_fix[layer], A.renorm,
                                     cs_p, ids_p, sc_p, fm, 1u << lane);
      else
        token_epilogue(row, E, k, c, A.eps_high[layer], A.t_fix[layer], A.renorm, cs_p, ids_p,
                       sc_p, fm, 1u << lane);
    }
    if (tok0 + warp * 32 < T) publish_group_masks(A, abs_layer, tok0 + warp * 32, fm, lane);
    team_barrier();   // every record of the tile is written
    if (tid == 0 && rt != A.withhold_tile) { __threadfence(); st_release(ready + rt, 1); }
  }
}

}  // namespace laser
#include "k1_router_tcp256.cuh"
namespace laser {

// Router role of one persistent block (256 threads): tiles first, first + step, ... < n_tiles of
// the launch's n_layers layers.  N: accumulator columns (64; 128 compiles but two such blocks do
// not fit one SM).
template <int N, int CL>
__device__ __forceinline__ void router_tcp_block(const RouteArgs& A, const CUtensorMap* map_h,
                                                 const CUtensorMap* map_w, int n_layers, int first,
                                                 int step, int n_tiles, unsigned char* dyn_smem) {
  constexpr int STAGES = tcp_stages<N>();
  constexpr int STAGE_BYTES = tc_stage_bytes<N>();
  constexpr int A_BYTES = kTcTileM * kTcSliceK * 2;
  constexpr uint32_t TMEM_COLS = 2 * N;   // two accumulators
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ uint32_t s_fm[4 * N];   // masks of the tile's four groups (see group_epilogue)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (warp >= 6) return;
  const int T = A.T, E = A.E, d = A.d;

  unsigned char* stages =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(dyn_smem) + 1023) & ~uintptr_t(1023));
  float* tile = reinterpret_cast<float*>(stages + (size_t)STAGES * STAGE_BYTES);
  float* bias_s = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(tile) + tcp_tile_bytes<N>());
  uint64_t* full = reinterpret_cast<uint64_t*>(bias_s + N);   // [STAGES] TMA landed
  uint64_t* empty = full + STAGES;                            // [STAGES] MMAs of the stage done
  uint64_t* acc_full = empty + STAGES;                        // [2] accumulator complete
  uint64_t* acc_empty = acc_full + 2;                         // [2] accumulator read by the team

  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < STAGES; ++s) { tc_mbar_init(full + s, 1); tc_mbar_init(empty + s, 1); }
    for (int a = 0; a < 2; ++a) { tc_mbar_init(acc_full + a, 1); tc_mbar_init(acc_empty + a, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  roles_barrier();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abort = &s_abort;
  const int nk = (d + kTcSliceK - 1) / kTcSliceK;
  auto give_up = [&]() {
    if (!*abort) { *abort = 1; if (A.status) atomicOr(A.status, 2); }
  };

  if (warp == 4) {
    if (lane == 0) {
      // ---- producer: one continuous stream of slices over all of the block's tiles
      long long it = 0;
      bool ok = true;
      for (int tile_id = first; tile_id < n_tiles && ok; tile_id += step) {
        const int layer = tile_id % n_layers, rt = tile_id / n_layers;
        const int abs_layer = A.layer0 + layer;
        const int row_h = abs_layer * T + rt * kTcTileM, row_w = abs_layer * E;
        for (int kc = 0; kc < nk; ++kc, ++it) {
          const int s = (int)(it % STAGES);
          const long long use = it / STAGES;
          if (use > 0 && !tc_mbar_wait(empty + s, (uint32_t)((use - 1) & 1), abort)) { ok = false; break; }
          unsigned char* sa = stages + (size_t)s * STAGE_BYTES;
          tc_mbar_expect_tx(full + s, (uint32_t)STAGE_BYTES);
          tma_load_2d(sa, map_h, full + s, kc * kTcSliceK, row_h);
          tma_load_2d(sa + A_BYTES, map_w, full + s, kc * kTcSliceK, row_w);
        }
      }
      if (!ok) {
        // gave up: make the others stop, then let the copies already issued land
        give_up();
        for (long long q = (it > STAGES ? it - STAGES : 0); q < it; ++q) {
          const long long start = clock64();
          while (!tc_mbar_try_wait(full + q % STAGES, (uint32_t)((q / STAGES) & 1)))
            if (clock64() - start > kTcWaitCycles) break;
        }
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      // ---- MMA issuer
      constexpr uint32_t idesc = tc_idesc(kTcTileM, N);
      long long it = 0;
      int j = 0;
      bool ok = true;
      for (int tile_id = first; tile_id < n_tiles && ok; tile_id += step, ++j) {
        const int a = j & 1;
        if (j >= 2 && !tc_mbar_wait(acc_empty + a, (uint32_t)(((j >> 1) - 1) & 1), abort)) { ok = false; break; }
        tc_fence_after();
        for (int kc = 0; kc < nk; ++kc, ++it) {
          const int s = (int)(it % STAGES);
          if (!tc_mbar_wait(full + s, (uint32_t)((it / STAGES) & 1), abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(stages + (size_t)s * STAGE_BYTES);
          const uint64_t adesc = tc_smem_desc(sa), bdesc = tc_smem_desc(sa + A_BYTES);
#pragma unroll
          for (int kk = 0; kk < kTcSliceK / 16; ++kk)
            tc_mma(tmem + (uint32_t)(a * N), adesc + 2 * kk, bdesc + 2 * kk, idesc,
                   (kc > 0 || kk > 0) ? 1u : 0u);
          tc_commit(empty + s);
        }
        if (ok) tc_commit(acc_full + a);
      }
      if (!ok) give_up();
    }
  } else {
    // ---- scoring team (see the second half of this function)
    if constexpr (N == 256)
      router_tcp256_team(A, n_layers, first, step, n_tiles, tmem, tile, bias_s, s_fm, acc_full,
                         acc_empty, abort);
    else
      router_tcp_team<N, CL>(A, n_layers, first, step, n_tiles, tmem, tile, bias_s, s_fm, acc_full,
                             acc_empty, abort);
  }
  __syncwarp();
  tc_fence_before();
  roles_barrier();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace laser
