// Template instances of the fused router + selection kernels (one group per file, see
// k12_launch.cuh).
#include "k12_launch.cuh"

namespace laser {

cudaError_t launch_splitk_e8(const RouteArgs& a, int n, cudaStream_t s) { return launch_k12_splitk_for_c<1, 4>(a, n, s); }
cudaError_t launch_splitk_e16(const RouteArgs& a, int n, cudaStream_t s) { return launch_k12_splitk_for_c<2, 4>(a, n, s); }

}  // namespace laser
