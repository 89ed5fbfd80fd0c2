// Template instances of the fused router + selection kernels (one group per file, see
// k12_launch.cuh).
#include "k12_launch.cuh"

namespace laser {

cudaError_t launch_warp_e256(const RouteArgs& a, int n, cudaStream_t s) { return launch_k12_for_c<32, 1, 1>(a, n, s); }

}  // namespace laser
