// Pipelined tile kernels (placeholder: no shape is planned onto this path yet).
#include "s2a_common.cuh"
#include "s2a_launch.h"

namespace s2a {

__device__ unsigned int g_error_word = 0;

TilePlan plan_tile(int, int, uint64_t, uint32_t) { return TilePlan{}; }

cudaError_t launch_tile(int, int, const TilePlan&, const TileArgs&, cudaStream_t) {
  return cudaErrorInvalidValue;
}

cudaError_t read_error_word(unsigned int* flags, bool clear) {
  cudaError_t e = cudaMemcpyFromSymbol(flags, g_error_word, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  if (clear) {
    unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_error_word, &zero, sizeof(unsigned int));
  }
  return e;
}

}  // namespace s2a
