// Host-side launch interfaces between the C-ABI entry points and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace s2a {

// Per-device host-side caches (attribute set-up, symbol addresses, SM counts) are tables of
// this many entries indexed by the CUDA device ordinal.
constexpr int kMaxDevices = 64;

enum { kGeluFwd = 0, kGeluBwd = 1, kSoftmaxFwd = 2, kSoftmaxBwd = 3, kSiluFwd = 4, kSiluBwd = 5 };

// Kernel-id predicates (GELU and SiLU share their code: "act" kernels).
__host__ __device__ constexpr bool is_act_fwd(int k) { return k == kGeluFwd || k == kSiluFwd; }
__host__ __device__ constexpr bool is_act_bwd(int k) { return k == kGeluBwd || k == kSiluBwd; }
__host__ __device__ constexpr bool is_fwd(int k) { return is_act_fwd(k) || k == kSoftmaxFwd; }
__host__ __device__ constexpr int act_of(int k) { return (k == kSiluFwd || k == kSiluBwd) ? 1 : 0; }

// One launch of a row-at-a-time kernel over rows [row0, row0 + n_rows) of a tensor.
// row0 * row_len must be even (whole code bytes).  `in` is x or grad_out, `out` is y or
// grad_in, both pointing at element 0 of the whole tensor; codes and meta likewise.
struct RowwiseArgs {
  const void* in;
  void* out;
  uint8_t* codes;  // written by the forward kernels, read by the backward kernels
  float* meta;     // likewise
  uint64_t row0;
  uint64_t n_rows;
  uint32_t row_len;
};

// bits: the code width (4 by default; 2 and 8 for the four kernels of the paper).  row0 * row_len
// must be a multiple of 8 / bits.
cudaError_t launch_rowwise(int kernel, int dt, const RowwiseArgs& a, cudaStream_t st, int bits = 4);

// ReLU with its 1-bit mask: in = x (forward) or grad_out (backward), out = y or grad_in.
cudaError_t launch_relu(bool fwd, int dt, const void* in, void* out, uint8_t* mask, uint64_t n, cudaStream_t st);

// GELU forward with one quantiser range for the whole tensor (two reads of x).  `scratch`
// is device memory of tensor_range_scratch_bytes(n) bytes, 8-byte aligned.
uint64_t tensor_range_scratch_bytes(uint64_t n);
cudaError_t launch_gelu_fwd_tensor_range(int dt, const void* x, void* y, uint8_t* codes, float* meta, float* scratch,
                                         uint64_t n, uint64_t n_rows, cudaStream_t st);

// The same three kernels with their scratch in a static device array of the library; no
// allocation anywhere.  n must not exceed tensor_range_static_max_elems().
uint64_t tensor_range_static_max_elems();
cudaError_t launch_gelu_fwd_tensor_range_static(int dt, const void* x, void* y, uint8_t* codes, float* meta,
                                                uint64_t n, uint64_t n_rows, cudaStream_t st);

// Channel Average Pooling (flat: n_out outputs, each the mean of r consecutive inputs; the
// backward spreads g / r) and the Low-Rank Prompt add.
cudaError_t launch_cap(bool fwd, int dt, const void* in, void* out, uint64_t n_out, uint32_t r, cudaStream_t st);
cudaError_t launch_lrp_fwd(int dt, const void* x, const float* A, const float* B, void* y, uint32_t batch,
                           uint32_t tokens, uint32_t channels, uint32_t rank, cudaStream_t st);

// ---------------------------------------------------------------- pipelined tiles
// A tile is `tile_rows` consecutive rows whose flat element span starts and ends on a
// multiple of 32 elements (128 / bits in general), so that its data and its code bytes can
// move with 16-byte bulk copies.  A plan with tile_rows == 0 means "no pipelined path for this shape".
enum { kVariantGeneric = 0, kVariantStream = 1, kVariantPairFixed = 2, kVariantAny = 3 };

struct TilePlan {
  uint32_t tile_rows;   // rows per tile (0: not applicable)
  uint32_t variant;     // kVariantGeneric / kVariantStream / kVariantPairFixed / kVariantAny
  uint32_t unit_lanes;  // lanes that cooperate on one row: 8, 16, 32 or 128
  uint32_t vec_elems;   // elements per shared-memory access: 2 (pair mode) or 16 bytes' worth
  uint32_t iters;       // accesses per lane per row kept in registers (0: streamed)
  uint32_t warps;       // consumer warps per CTA (one more warp drives the copies)
  uint32_t stages;      // tiles resident in shared memory per CTA
  uint32_t smem_bytes;  // dynamic shared memory per CTA
  uint32_t grid;        // CTAs launched
  uint64_t n_tiles;     // full tiles covered; remaining rows go to the row-at-a-time path
  uint32_t overlap_launch;  // 1: launched with programmatic stream serialization
  uint32_t bits;        // code width of Eq. 8: 4, or 2 / 8 (GELU rows of whole 16-byte vectors)
  uint32_t rows_per_group;  // rows a unit takes together (the kernel's WORK::rows_per_group); divides tile_rows
  uint32_t spread_units;    // 1: the sub-warp units of a warp take groups tile_groups / (units per warp) apart
  uint32_t ragged_codes;    // 1: a tile's code bytes need not start on a 16-byte boundary of the code tensor
};

struct TileArgs {
  const void* in;
  void* out;
  uint8_t* codes;
  float* meta;
  uint32_t row_len;
  uint64_t n_tiles;
};

// Chooses the launch shape for (kernel, dt, row_len, n_rows) on the current device.
TilePlan plan_tile(int kernel, int dt, uint64_t n_rows, uint32_t row_len, int bits = 4);
cudaError_t launch_tile(int kernel, int dt, const TilePlan& p, const TileArgs& a, cudaStream_t st);

// Reads (and optionally clears) the per-device error word the pipelined kernels set
// when a bounded wait runs out.  Synchronises the device.
cudaError_t read_error_word(unsigned int* flags, bool clear);

// Launches the bounded wait's self-test (a wait that is meant to run out after 2 ms).
cudaError_t launch_wait_expiry_probe(cudaStream_t st);
// Counts the neighbouring binary32 arguments in [-150, 1] at which the hardware's approximate 2^x decreases.
cudaError_t count_exp2_out_of_order(unsigned long long* count, cudaStream_t st);

}  // namespace s2a
