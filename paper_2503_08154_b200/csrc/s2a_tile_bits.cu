// Instantiations of the pipelined tile kernel for Eq. 8 at 2 and 8 bits.
#include "s2a_tile.cuh"

namespace s2a {

cudaError_t launch_tile_bits(int kernel, int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st) {
  const TileKernelArgs& ka = *(const TileKernelArgs*)kernel_args;
  if (kernel == kGeluFwd) return launch_tile_bits_kernel<kGeluFwd>(dt, p, ka, st);
  if (kernel == kGeluBwd) return launch_tile_bits_kernel<kGeluBwd>(dt, p, ka, st);
  if (kernel == kSoftmaxFwd) return launch_tile_bits_kernel<kSoftmaxFwd>(dt, p, ka, st);
  if (kernel == kSoftmaxBwd) return launch_tile_bits_kernel<kSoftmaxBwd>(dt, p, ka, st);
  return cudaErrorInvalidValue;
}

}  // namespace s2a
