// Instantiations of the fixed-width softmax kernels for the attention widths other than
// 197 and 257 (49, 50, 145, 196, 198, 577, 1025).
#include "s2a_tile.cuh"

namespace s2a {

cudaError_t launch_tile_pair_widths(int kernel, int dt, const TilePlan& p, const void* kernel_args, cudaStream_t st) {
  const TileKernelArgs& ka = *(const TileKernelArgs*)kernel_args;
  if (kernel == kSoftmaxFwd) return launch_tile_pair_widths_kernel<kSoftmaxFwd>(dt, p, ka, st);
  if (kernel == kSoftmaxBwd) return launch_tile_pair_widths_kernel<kSoftmaxBwd>(dt, p, ka, st);
  return cudaErrorInvalidValue;
}

}  // namespace s2a
