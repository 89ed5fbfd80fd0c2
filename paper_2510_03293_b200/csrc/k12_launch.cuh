// Launch helpers of the fused router + selection kernels, and the per-shape launchers that the
// instantiation files (k12_inst_*.cu) define, one group of template instances per file so
// that the library builds in parallel.
#pragma once
#include "k12_fused.cuh"

namespace laser {

// shared memory the selection role needs in a launch
inline size_t selection_smem(const RouteArgs& a) {
  const size_t b = k2_smem_bytes(a.E, a.c, a.k);
  const size_t f = a.fuse_dispatch ? k2_fused_dispatch_bytes(a.E, a.k) : 0;
  return b > f ? b : f;
}

template <int NT, int MT, int KU, int CMAX>
cudaError_t launch_k12(const RouteArgs& a, int n_layers, cudaStream_t s) {
  size_t smem = router_smem_bytes(NT, MT);
  const size_t smem2 = selection_smem(a);
  if (smem2 > smem) smem = smem2;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k12_route_select<NT, MT, KU, CMAX>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  constexpr int RR = router_rows<NT, MT>();
  const unsigned router_tiles = (unsigned)((a.T + RR - 1) / RR);
  k12_route_select<NT, MT, KU, CMAX>
      <<<n_layers * (1 + router_tiles), kK2Threads, smem, s>>>(a, n_layers);
  return cudaGetLastError();
}

// The selection sorts CMAX >= c candidate keys in registers; pick the smallest network.
template <int NT, int MT, int KU>
cudaError_t launch_k12_for_c(const RouteArgs& a, int n_layers, cudaStream_t s) {
  constexpr int EP = NT * 8;
  if (EP >= 4 && a.c <= 4) return launch_k12<NT, MT, KU, 4>(a, n_layers, s);
  if (EP >= 8 && a.c <= 8) return launch_k12<NT, MT, KU, 8>(a, n_layers, s);
  if (EP >= 16 && a.c <= 16) return launch_k12<NT, MT, KU, (EP >= 16 ? 16 : 8)>(a, n_layers, s);
  return launch_k12<NT, MT, KU, (EP >= 32 ? 32 : EP)>(a, n_layers, s);
}

template <int N, int CMAX>
cudaError_t launch_k12_tc(const RouteArgs& a, int n_layers, const CUtensorMap& mh,
                          const CUtensorMap& mw, cudaStream_t s) {
  size_t smem = tc_smem_bytes<N>();
  const size_t smem2 = selection_smem(a);
  if (smem2 > smem) smem = smem2;
  cudaError_t e = cudaFuncSetAttribute(k12_route_select_tc<N, CMAX>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const unsigned tiles = (unsigned)((a.T + kTcTileM - 1) / kTcTileM);
  k12_route_select_tc<N, CMAX><<<n_layers * (1 + tiles), kK2Threads, smem, s>>>(a, n_layers, mh, mw);
  return cudaGetLastError();
}

// Persistent form (N = 64 or 256): router_blocks blocks walk all tiles of the launch.
template <int N, int CMAX>
cudaError_t launch_k12_tcp(const RouteArgs& a, int n_layers, int router_blocks,
                           const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s) {
  size_t smem = tcp_smem_bytes<N>();
  const size_t smem2 = selection_smem(a);
  if (smem2 > smem) smem = smem2;
  cudaError_t e = cudaFuncSetAttribute(k12_route_select_tcp<N, CMAX>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int n_tiles = n_layers * ((a.T + kTcTileM - 1) / kTcTileM);
  if (router_blocks > n_tiles) router_blocks = n_tiles;
  k12_route_select_tcp<N, CMAX>
      <<<n_layers + router_blocks, kK2Threads, smem, s>>>(a, n_layers, n_tiles, mh, mw);
  return cudaGetLastError();
}

template <int N>
cudaError_t launch_k12_tcp_for_c(const RouteArgs& a, int n_layers, int router_blocks,
                                 const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s) {
  if (a.c <= 4) return launch_k12_tcp<N, 4>(a, n_layers, router_blocks, mh, mw, s);
  if (a.c <= 8) return launch_k12_tcp<N, 8>(a, n_layers, router_blocks, mh, mw, s);
  if (a.c <= 16) return launch_k12_tcp<N, 16>(a, n_layers, router_blocks, mh, mw, s);
  return launch_k12_tcp<N, 32>(a, n_layers, router_blocks, mh, mw, s);
}

template <int N>
cudaError_t launch_k12_tc_for_c(const RouteArgs& a, int n_layers, const CUtensorMap& mh,
                                const CUtensorMap& mw, cudaStream_t s) {
  if (a.c <= 4) return launch_k12_tc<N, 4>(a, n_layers, mh, mw, s);
  if (a.c <= 8) return launch_k12_tc<N, 8>(a, n_layers, mh, mw, s);
  if (a.c <= 16) return launch_k12_tc<N, 16>(a, n_layers, mh, mw, s);
  return launch_k12_tc<N, 32>(a, n_layers, mh, mw, s);
}

// ---- split-K router for calls with few tokens ---------------------------------------------
template <int NT, int KU, int CMAX>
cudaError_t launch_k12_splitk(const RouteArgs& a, int n_layers, cudaStream_t s) {
  size_t smem = router_splitk_smem_bytes(NT);
  const size_t smem2 = selection_smem(a);
  if (smem2 > smem) smem = smem2;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k12_route_select_splitk<NT, KU, CMAX>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const unsigned tiles = (unsigned)((a.T + 15) / 16);
  if (a.cluster_tiles > 0) {
    // one cluster per layer: the selection block and the layer's router tiles
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_layers * (1 + tiles));
    cfg.blockDim = dim3(kK2Threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1 + tiles;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k12_route_select_splitk<NT, KU, CMAX>, a, n_layers);
  }
  k12_route_select_splitk<NT, KU, CMAX>
      <<<n_layers * (1 + tiles), kK2Threads, smem, s>>>(a, n_layers);
  return cudaGetLastError();
}

template <int NT, int KU>
cudaError_t launch_k12_splitk_for_c(const RouteArgs& a, int n_layers, cudaStream_t s) {
  constexpr int EP = NT * 8;
  if (a.c <= 4) return launch_k12_splitk<NT, KU, 4>(a, n_layers, s);
  if (a.c <= 8) return launch_k12_splitk<NT, KU, 8>(a, n_layers, s);
  if (a.c <= 16) return launch_k12_splitk<NT, KU, (EP >= 16 ? 16 : 8)>(a, n_layers, s);
  return launch_k12_splitk<NT, KU, (EP >= 32 ? 32 : EP)>(a, n_layers, s);
}


// defined in k12_inst_*.cu
cudaError_t launch_warp_e8(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_warp_e16(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_warp_e32(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_warp_e64(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_warp_e128(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_warp_e256(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e8(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e16(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e32(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e64(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e128(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_splitk_e256(const RouteArgs& a, int n_layers, cudaStream_t s);
cudaError_t launch_tc_n64(const RouteArgs& a, int n_layers, const CUtensorMap& mh,
                          const CUtensorMap& mw, cudaStream_t s);
cudaError_t launch_tc_n128(const RouteArgs& a, int n_layers, const CUtensorMap& mh,
                           const CUtensorMap& mw, cudaStream_t s);
cudaError_t launch_tc_n256(const RouteArgs& a, int n_layers, const CUtensorMap& mh,
                           const CUtensorMap& mw, cudaStream_t s);
cudaError_t launch_tcp_n256(const RouteArgs& a, int n_layers, int router_blocks,
                            const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s);
cudaError_t launch_tcp_n64(const RouteArgs& a, int n_layers, int router_blocks,
                           const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s);


}  // namespace laser
