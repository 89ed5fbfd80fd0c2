// Template instances of the fused router + selection kernels (one group per file, see
// k12_launch.cuh).
#include "k12_launch.cuh"

namespace laser {

cudaError_t launch_tcp_n64(const RouteArgs& a, int n, int router_blocks, const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s) { return launch_k12_tcp_for_c<64>(a, n, router_blocks, mh, mw, s); }

}  // namespace laser
