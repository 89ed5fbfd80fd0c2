// Template instances of the fused router + selection kernels (one group per file, see
// k12_launch.cuh).
#include "k12_launch.cuh"

namespace laser {

cudaError_t launch_tc_n256(const RouteArgs& a, int n, const CUtensorMap& mh, const CUtensorMap& mw, cudaStream_t s) { return launch_k12_tc_for_c<256>(a, n, mh, mw, s); }

}  // namespace laser
