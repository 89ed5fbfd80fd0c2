// One launch for the router and the ordered selection.  The first n_layers blocks take the
// selection role (one per layer); every other block routes one tile of router_rows tokens of
// one layer and then publishes a ready flag for it.  Router blocks are numbered token-major
// (the layer index varies fastest), so all layers advance together and each selection block
// trails the router by about one tile instead of starting after the last router block.
// Router blocks never wait, and there are far fewer selection blocks than the GPU can hold,
// so the waits of the selection role always end; they are bounded all the same.
#pragma once
#include "k1_router.cuh"
#include "k2_select.cuh"
#include "k1_router_tc.cuh"
#include "k1_router_tcp.cuh"

namespace laser {

constexpr int kRouterWarps = kK2Threads / 32;

template <int NT, int MT>
__host__ __device__ constexpr int router_rows() { return kRouterWarps * MT * 16; }

// logits tile of the block, then one mask scratch of NT * 8 words per warp (see group_epilogue)
__host__ __device__ inline size_t router_tile_bytes(int NT, int MT) {
  return sizeof(float) * kRouterWarps * MT * 16 * (NT * 8 + 1);
}
__host__ __device__ inline size_t router_smem_bytes(int NT, int MT) {
  return router_tile_bytes(NT, MT) + (NT * 8 > 32 ? sizeof(uint32_t) * kRouterWarps * NT * 8 : 0);
}

template <int NT, int MT, int KU, int CMAX>
__global__ void __launch_bounds__(kK2Threads) k12_route_select(const RouteArgs A, int n_layers) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  constexpr int RR = router_rows<NT, MT>();
  constexpr int LDS = NT * 8 + 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if ((int)blockIdx.x < n_layers) {
    const int layer = A.layer0 + blockIdx.x;
    const int* ready = reinterpret_cast<const int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready);
    k2_block<CMAX, (NT * 8 <= 32)>(A, layer, dyn_smem, ready, RR);
    return;
  }
  const int b = blockIdx.x - n_layers;
  const int local_layer = b % n_layers;
  const int rt = b / n_layers;
  float* tiles = reinterpret_cast<float*>(dyn_smem);
  uint32_t* fm = reinterpret_cast<uint32_t*>(dyn_smem + router_tile_bytes(NT, MT)) + warp * (NT * 8);
  const long long tok0 = (long long)rt * RR + (long long)warp * (MT * 16);
  if (tok0 < A.T) router_warp<NT, MT, KU>(A, local_layer, tok0, tiles + (size_t)warp * (MT * 16) * LDS, lane);
  if (MT == 2) {
    // a warp's 32 rows are one group: no block-wide hand-over needed
    if (tok0 < A.T)
      group_epilogue(A, local_layer, tok0, tiles + (size_t)warp * 32 * LDS, LDS, lane, fm);
  } else {
    __syncthreads();
    const long long gtok0 = (long long)rt * RR + (long long)warp * 32;
    if (warp * 32 < RR && gtok0 < A.T)
      group_epilogue(A, local_layer, gtok0, tiles + (size_t)warp * 32 * LDS, LDS, lane, fm);
  }
  __syncthreads();
  if (tid == 0 && rt != A.withhold_tile) {
    int* ready = reinterpret_cast<int*>(A.ws + (size_t)(A.layer0 + local_layer) * A.ws_ls +
                                        A.lay.ready);
    __threadfence();
    st_release(ready + rt, 1);
  }
}

// The same launch shape with the split-K router for calls with few tokens: every router block
// routes 16 tokens.
template <int NT, int KU, int CMAX>
__global__ void __launch_bounds__(kK2Threads)
k12_route_select_splitk(const RouteArgs A, int n_layers) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  if (A.cluster_tiles > 0) {
    // Few tiles per layer: the launch is one cluster per layer (rank 0 selects, ranks 1.. route
    // one tile each).  The routers never wait, so every block reaches the cluster barrier, and
    // the selection starts behind it with all records in place: no flags, no polling.
    const int cs = A.cluster_tiles + 1;
    const int rank = (int)blockIdx.x % cs, local_layer = (int)blockIdx.x / cs;
    if (rank > 0) {
      router_splitk_block<NT, KU>(A, local_layer, rank - 1, reinterpret_cast<float*>(dyn_smem));
      __threadfence();
    }
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (rank == 0)
      k2_block<CMAX, (NT * 8 <= 32)>(A, A.layer0 + local_layer, dyn_smem, nullptr, 16);
    return;
  }
  if ((int)blockIdx.x < n_layers) {
    const int layer = A.layer0 + blockIdx.x;
    const int* ready = reinterpret_cast<const int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready);
    k2_block<CMAX, (NT * 8 <= 32)>(A, layer, dyn_smem, ready, 16);
    return;
  }
  const int b = blockIdx.x - n_layers;
  const int local_layer = b % n_layers;
  const int rt = b / n_layers;
  router_splitk_block<NT, KU>(A, local_layer, rt, reinterpret_cast<float*>(dyn_smem));
  __syncthreads();
  if (threadIdx.x == 0 && rt != A.withhold_tile) {
    int* ready = reinterpret_cast<int*>(A.ws + (size_t)(A.layer0 + local_layer) * A.ws_ls +
                                        A.lay.ready);
    __threadfence();
    st_release(ready + rt, 1);
  }
}

// The same launch shape with the tensor-memory router (E > 32): the first n_layers blocks
// select, every other block routes one tile of 128 tokens.
template <int N, int CMAX>
__global__ void __launch_bounds__(kK2Threads, tc_min_blocks<N>())
k12_route_select_tc(const RouteArgs A, int n_layers, const __grid_constant__ CUtensorMap map_h,
                    const __grid_constant__ CUtensorMap map_w) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  if ((int)blockIdx.x < n_layers) {
    const int layer = A.layer0 + blockIdx.x;
    const int* ready = reinterpret_cast<const int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready);
    // A resident block that never gives up its right to allocate tensor memory keeps router
    // blocks of this kernel off its SM.  The selection role needs no tensor memory and, for the
    // rule's own update order, is mostly waiting, so it gives the right up at once and router
    // blocks share its SM.
    if (threadIdx.x < 32)
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    k2_block<CMAX, false>(A, layer, dyn_smem, ready, kTcTileM);
    return;
  }
  const int b = blockIdx.x - n_layers;
  const int local_layer = b % n_layers;
  const int rt = b / n_layers;
  const bool done =
      router_tc_block<N, (CMAX < 8 ? 8 : CMAX)>(A, &map_h, &map_w, local_layer, rt, dyn_smem);
  // router_tc_block ends with a block barrier after the last record was written; a tile whose
  // own waits ran out wrote no records and says so (-1), which aborts the layer's selection
  if (threadIdx.x == 0 && rt != A.withhold_tile) {
    int* ready = reinterpret_cast<int*>(A.ws + (size_t)(A.layer0 + local_layer) * A.ws_ls +
                                        A.lay.ready);
    __threadfence();
    st_release(ready + rt, done ? 1 : -1);
  }
}

// The persistent form of the tensor-memory router (E <= 64, or 128 < E <= 256 with c <= 16): the first n_layers blocks select,
// every other block walks the tiles b, b + P, ... of all layers (tile id = tile index * n_layers
// + layer).
template <int N, int CMAX>
__global__ void __launch_bounds__(kK2Threads, N <= 64 ? 2 : 1)
k12_route_select_tcp(const RouteArgs A, int n_layers, int n_tiles,
                     const __grid_constant__ CUtensorMap map_h,
                     const __grid_constant__ CUtensorMap map_w) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  if ((int)blockIdx.x < n_layers) {
    const int layer = A.layer0 + blockIdx.x;
    const int* ready = reinterpret_cast<const int*>(A.ws + (size_t)layer * A.ws_ls + A.lay.ready);
    if (threadIdx.x < 32)   // the selection needs no tensor memory: router blocks share its SM
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    k2_block<CMAX, false>(A, layer, dyn_smem, ready, kTcTileM);
    return;
  }
  router_tcp_block<N, (CMAX < 8 ? 8 : CMAX)>(A, &map_h, &map_w, n_layers,
                                             (int)blockIdx.x - n_layers,
                                             (int)gridDim.x - n_layers, n_tiles, dyn_smem);
}

}  // namespace laser
