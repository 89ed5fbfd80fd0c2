// Template instances of the fused router + selection kernels (one group per file, see
// k12_launch.cuh).
#include "k12_launch.cuh"

namespace laser {

// 256 accumulator columns, candidate lists of at most 16 (the team's list length)
cudaError_t launch_tcp_n256(const RouteArgs& a, int n, int router_blocks, const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s) {
  if (a.c <= 4) return launch_k12_tcp<256, 4>(a, n, router_blocks, mh, mw, s);
  if (a.c <= 8) return launch_k12_tcp<256, 8>(a, n, router_blocks, mh, mw, s);
  return launch_k12_tcp<256, 16>(a, n, router_blocks, mh, mw, s);
}

}  // namespace laser
