// Instantiations of the pipelined tile kernel for s2a_gelu_fwd.
#include "s2a_tile.cuh"

namespace s2a {

cudaError_t launch_tile_gelu_fwd(int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st) {
  return launch_tile_kernel<kGeluFwd>(dt, p, *(const TileKernelArgs*)kernel_args, st);
}

}  // namespace s2a
