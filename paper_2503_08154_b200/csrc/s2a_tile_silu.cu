// Instantiations of the pipelined tile kernel for s2a_silu_fwd and s2a_silu_bwd.
#include "s2a_tile.cuh"

namespace s2a {

cudaError_t launch_tile_silu_fwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st) {
  return launch_tile_kernel<kSiluFwd>(dt, p, *(const TileKernelArgs*)kernel_args, st);
}

cudaError_t launch_tile_silu_bwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st) {
  return launch_tile_kernel<kSiluBwd>(dt, p, *(const TileKernelArgs*)kernel_args, st);
}

}  // namespace s2a
