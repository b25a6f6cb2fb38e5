// extern "C" entry points of libs2a.so: argument checks, choice of kernel path, launch.
#include <stdio.h>
#include <string.h>

#include "../../include/s2a.h"
#include "s2a_common.cuh"
#include "s2a_launch.h"

namespace {

using namespace s2a;

bool misaligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) != 0; }

int check_args(const void* a, const void* b, const void* codes, const void* meta, size_t n,
               size_t row_len, int dt) {
  if (dt != S2A_F32 && dt != S2A_BF16) return S2A_ERR_DTYPE;
  if (row_len == 0 || row_len > 0x7fffffffull || n % row_len != 0) return S2A_ERR_SHAPE;
  if (n == 0) return S2A_OK;
  if (!a || !b || !codes || !meta) return S2A_ERR_NULL;
  if (misaligned(a, 16) || misaligned(b, 16) || misaligned(codes, 16) || misaligned(meta, 8))
    return S2A_ERR_ALIGN;
  // in-place (a == b) is fine: every element, and every row, is read before it is written;
  // an output that merely overlaps its input would be overwritten while still unread
  if (a != b) {
    const uintptr_t bytes = (uintptr_t)n * (dt == S2A_F32 ? 4u : 2u);
    const uintptr_t pa = (uintptr_t)a, pb = (uintptr_t)b;
    if (pa < pb + bytes && pb < pa + bytes) return S2A_ERR_OVERLAP;
  }
  return S2A_OK;
}

// Full tiles go to the pipelined kernel, whatever rows remain to the row-at-a-time one.
int run(int kernel, const void* in, void* out, uint8_t* codes, float* meta, size_t n,
        size_t row_len, int dt, void* stream) {
  int rc = check_args(in, out, codes, meta, n, row_len, dt);
  if (rc != S2A_OK || n == 0) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const uint64_t n_rows = n / row_len;
  TilePlan p = plan_tile(kernel, dt, n_rows, (uint32_t)row_len);
  uint64_t done_rows = 0;
  // the pipelined path moves metadata with 16-byte bulk copies
  if (p.tile_rows != 0 && p.n_tiles != 0 && !misaligned(meta, 16)) {
    TileArgs ta{in, out, codes, meta, (uint32_t)row_len, p.n_tiles};
    if (launch_tile(kernel, dt, p, ta, st) != cudaSuccess) return S2A_ERR_CUDA;
    done_rows = p.n_tiles * p.tile_rows;
  }
  if (done_rows < n_rows) {
    RowwiseArgs ra{in, out, codes, meta, done_rows, n_rows - done_rows, (uint32_t)row_len};
    if (launch_rowwise(kernel, dt, ra, st) != cudaSuccess) return S2A_ERR_CUDA;
  }
  return S2A_OK;
}

}  // namespace

extern "C" {

size_t s2a_codes_bytes(size_t n_elems) { return (n_elems + 1) / 2; }

size_t s2a_meta_bytes(size_t n_elems, size_t row_len) {
  return row_len == 0 ? 0 : (n_elems / row_len) * 2 * sizeof(float);
}

const char* s2a_status_string(int status) {
  switch (status) {
    case S2A_OK: return "S2A_OK";
    case S2A_ERR_NULL: return "S2A_ERR_NULL: a required pointer is NULL";
    case S2A_ERR_SHAPE: return "S2A_ERR_SHAPE: row_len is 0 or does not divide n_elems";
    case S2A_ERR_ALIGN: return "S2A_ERR_ALIGN: data/codes need 16-byte, meta 8-byte alignment";
    case S2A_ERR_DTYPE: return "S2A_ERR_DTYPE: dt must be S2A_F32 or S2A_BF16";
    case S2A_ERR_CUDA: return "S2A_ERR_CUDA: the CUDA runtime refused the launch";
    case S2A_ERR_DEVICE: return "S2A_ERR_DEVICE: a kernel gave up on a bounded wait";
    case S2A_ERR_TOO_LARGE:
      return "S2A_ERR_TOO_LARGE: n_elems exceeds the built-in scratch of the allocation-free entry point "
             "(536,870,912 elements); use s2a_gelu_fwd_tensor_range with your own scratch";
    case S2A_ERR_OVERLAP: return "S2A_ERR_OVERLAP: the output overlaps the input without being the same tensor";
    default: return "unknown s2a status";
  }
}

int s2a_gelu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                 size_t row_len, int dt, void* cuda_stream) {
  return run(kGeluFwd, x, y, codes, meta, n_elems, row_len, dt, cuda_stream);
}

int s2a_gelu_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                 size_t n_elems, size_t row_len, int dt, void* cuda_stream) {
  return run(kGeluBwd, grad_out, grad_in, const_cast<uint8_t*>(codes), const_cast<float*>(meta),
             n_elems, row_len, dt, cuda_stream);
}

int s2a_softmax_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                    size_t row_len, int dt, void* cuda_stream) {
  return run(kSoftmaxFwd, x, y, codes, meta, n_elems, row_len, dt, cuda_stream);
}

int s2a_softmax_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                    size_t n_elems, size_t row_len, int dt, void* cuda_stream) {
  return run(kSoftmaxBwd, grad_out, grad_in, const_cast<uint8_t*>(codes),
             const_cast<float*>(meta), n_elems, row_len, dt, cuda_stream);
}

static int run_cap(bool fwd, const void* in, void* out, size_t n_rows, size_t channels, size_t r, int dt,
                   void* stream) {
  if (dt != S2A_F32 && dt != S2A_BF16) return S2A_ERR_DTYPE;
  if (r == 0 || r > 0x7fffffffull || channels % r != 0) return S2A_ERR_SHAPE;
  if (n_rows * channels == 0) return S2A_OK;
  if (!in || !out) return S2A_ERR_NULL;
  if (misaligned(in, 16) || misaligned(out, 16)) return S2A_ERR_ALIGN;
  return launch_cap(fwd, dt, in, out, n_rows * (channels / r), (uint32_t)r, (cudaStream_t)stream) == cudaSuccess
             ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_cap_fwd(const void* x, void* y, size_t n_rows, size_t channels, size_t r, int dt, void* cuda_stream) {
  return run_cap(true, x, y, n_rows, channels, r, dt, cuda_stream);
}

int s2a_cap_bwd(const void* grad_out, void* grad_in, size_t n_rows, size_t channels, size_t r, int dt,
                void* cuda_stream) {
  return run_cap(false, grad_out, grad_in, n_rows, channels, r, dt, cuda_stream);
}

int s2a_lrp_fwd(const void* x, const float* A, const float* B, void* y, size_t batch, size_t tokens,
                size_t channels, size_t rank, int dt, void* cuda_stream) {
  if (dt != S2A_F32 && dt != S2A_BF16) return S2A_ERR_DTYPE;
  if (batch > 0xffffffffull || tokens > 0xffffffffull || channels > 0xffffffffull || rank > 0xffffffffull)
    return S2A_ERR_SHAPE;
  if (batch * tokens * channels == 0) return S2A_OK;
  if (!x || !y || (rank > 0 && (!A || !B))) return S2A_ERR_NULL;
  if (misaligned(x, 16) || misaligned(y, 16) || misaligned(A, 4) || misaligned(B, 4)) return S2A_ERR_ALIGN;
  return launch_lrp_fwd(dt, x, A, B, y, (uint32_t)batch, (uint32_t)tokens, (uint32_t)channels, (uint32_t)rank,
                        (cudaStream_t)cuda_stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_silu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len, int dt,
                 void* cuda_stream) {
  return run(kSiluFwd, x, y, codes, meta, n_elems, row_len, dt, cuda_stream);
}

int s2a_silu_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in, size_t n_elems,
                 size_t row_len, int dt, void* cuda_stream) {
  return run(kSiluBwd, grad_out, grad_in, const_cast<uint8_t*>(codes), const_cast<float*>(meta), n_elems, row_len,
             dt, cuda_stream);
}

size_t s2a_tensor_range_scratch_bytes(size_t n_elems) { return (size_t)tensor_range_scratch_bytes(n_elems); }

int s2a_gelu_fwd_tensor_range(const void* x, void* y, uint8_t* codes, float* meta, void* scratch,
                              size_t n_elems, size_t row_len, int dt, void* cuda_stream) {
  int rc = check_args(x, y, codes, meta, n_elems, row_len, dt);
  if (rc != S2A_OK || n_elems == 0) return rc;
  if (!scratch) return S2A_ERR_NULL;
  if (misaligned(scratch, 8)) return S2A_ERR_ALIGN;
  return launch_gelu_fwd_tensor_range(dt, x, y, codes, meta, (float*)scratch, n_elems, n_elems / row_len,
                                      (cudaStream_t)cuda_stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

size_t s2a_tensor_range_static_max_elems(void) { return (size_t)tensor_range_static_max_elems(); }

int s2a_gelu_fwd_tensor_range_static(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                                     size_t row_len, int dt, void* cuda_stream) {
  int rc = check_args(x, y, codes, meta, n_elems, row_len, dt);
  if (rc != S2A_OK || n_elems == 0) return rc;
  if (n_elems > tensor_range_static_max_elems()) return S2A_ERR_TOO_LARGE;
  return launch_gelu_fwd_tensor_range_static(dt, x, y, codes, meta, n_elems, n_elems / row_len,
                                             (cudaStream_t)cuda_stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

size_t s2a_mask_bytes(size_t n_elems) { return (n_elems + 7) / 8; }

static int run_relu(bool fwd, const void* in, void* out, uint8_t* mask, size_t n, int dt, void* stream) {
  if (dt != S2A_F32 && dt != S2A_BF16) return S2A_ERR_DTYPE;
  if (n == 0) return S2A_OK;
  if (!in || !out || !mask) return S2A_ERR_NULL;
  if (misaligned(in, 16) || misaligned(out, 16)) return S2A_ERR_ALIGN;
  return launch_relu(fwd, dt, in, out, mask, n, (cudaStream_t)stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_relu_fwd(const void* x, void* y, uint8_t* mask, size_t n_elems, int dt, void* cuda_stream) {
  return run_relu(true, x, y, mask, n_elems, dt, cuda_stream);
}

int s2a_relu_bwd(const void* grad_out, const uint8_t* mask, void* grad_in, size_t n_elems, int dt,
                 void* cuda_stream) {
  return run_relu(false, grad_out, grad_in, const_cast<uint8_t*>(mask), n_elems, dt, cuda_stream);
}

size_t s2a_codes_bytes_bits(size_t n_elems, int bits) {
  return (bits == 2 || bits == 4 || bits == 8) ? (n_elems * (size_t)bits + 7) / 8 : 0;
}

// General code width: 4 goes to the ordinary entry points.  At 2 and 8 bits the GELU
// kernels have a pipelined form for rows of whole 16-byte vectors; everything else, and
// the rows left over, run row at a time.
static int run_bits(int kernel, const void* in, void* out, uint8_t* codes, float* meta, size_t n, size_t row_len,
                    int bits, int dt, void* stream) {
  if (bits == 4) return run(kernel, in, out, codes, meta, n, row_len, dt, stream);
  if (bits != 2 && bits != 8) return S2A_ERR_SHAPE;
  int rc = check_args(in, out, codes, meta, n, row_len, dt);
  if (rc != S2A_OK || n == 0) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const uint64_t n_rows = n / row_len;
  uint64_t done_rows = 0;
  TilePlan p = plan_tile(kernel, dt, n_rows, (uint32_t)row_len, bits);
  if (p.tile_rows != 0 && p.n_tiles != 0 && !misaligned(meta, 16)) {
    TileArgs ta{in, out, codes, meta, (uint32_t)row_len, p.n_tiles};
    if (launch_tile(kernel, dt, p, ta, st) != cudaSuccess) return S2A_ERR_CUDA;
    done_rows = p.n_tiles * p.tile_rows;
  }
  if (done_rows < n_rows) {
    RowwiseArgs ra{in, out, codes, meta, done_rows, n_rows - done_rows, (uint32_t)row_len};
    if (launch_rowwise(kernel, dt, ra, st, bits) != cudaSuccess) return S2A_ERR_CUDA;
  }
  return S2A_OK;
}

int s2a_gelu_fwd_bits(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len,
                      int bits, int dt, void* cuda_stream) {
  return run_bits(kGeluFwd, x, y, codes, meta, n_elems, row_len, bits, dt, cuda_stream);
}
int s2a_gelu_bwd_bits(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in, size_t n_elems,
                      size_t row_len, int bits, int dt, void* cuda_stream) {
  return run_bits(kGeluBwd, grad_out, grad_in, const_cast<uint8_t*>(codes), const_cast<float*>(meta), n_elems,
                  row_len, bits, dt, cuda_stream);
}
int s2a_softmax_fwd_bits(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len,
                         int bits, int dt, void* cuda_stream) {
  return run_bits(kSoftmaxFwd, x, y, codes, meta, n_elems, row_len, bits, dt, cuda_stream);
}
int s2a_softmax_bwd_bits(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                         size_t n_elems, size_t row_len, int bits, int dt, void* cuda_stream) {
  return run_bits(kSoftmaxBwd, grad_out, grad_in, const_cast<uint8_t*>(codes), const_cast<float*>(meta), n_elems,
                  row_len, bits, dt, cuda_stream);
}

int s2a_device_error(unsigned int* flags, int clear) {
  if (!flags) return S2A_ERR_NULL;
  return read_error_word(flags, clear != 0) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_selftest_wait_expiry(void* cuda_stream) {
  return launch_wait_expiry_probe((cudaStream_t)cuda_stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_selftest_exp2_monotone(unsigned long long* out_of_order, void* cuda_stream) {
  if (!out_of_order) return S2A_ERR_NULL;
  return count_exp2_out_of_order(out_of_order, (cudaStream_t)cuda_stream) == cudaSuccess ? S2A_OK : S2A_ERR_CUDA;
}

int s2a_describe_plan(int kernel, size_t n_elems, size_t row_len, int dt, char* out, size_t cap) {
  if (!out || cap == 0) return S2A_ERR_NULL;
  out[0] = 0;
  if (kernel < 0 || kernel > 5) return S2A_ERR_SHAPE;
  if (dt != S2A_F32 && dt != S2A_BF16) return S2A_ERR_DTYPE;
  if (row_len == 0 || row_len > 0x7fffffffull || n_elems % row_len != 0) return S2A_ERR_SHAPE;
  const uint64_t n_rows = n_elems / row_len;
  TilePlan p = plan_tile(kernel, dt, n_rows, (uint32_t)row_len);
  if (p.tile_rows == 0 || p.n_tiles == 0) {
    snprintf(out, cap, "rowwise rows=%llu", (unsigned long long)n_rows);
  } else {
    snprintf(out, cap,
             "tile variant=%s rows/tile=%u unit=%u vec=%u iters=%u warps=%u stages=%u smem=%u grid=%u "
             "group=%u spread=%u ragged_codes=%u tiles=%llu tail_rows=%llu",
             p.variant == kVariantStream ? "stream" : (p.variant == kVariantPairFixed ? "pair-fixed" : (p.variant == kVariantAny ? "any-length" : "generic")),
             p.tile_rows, p.unit_lanes, p.vec_elems, p.iters, p.warps, p.stages, p.smem_bytes,
             p.grid, p.rows_per_group, p.spread_units, p.ragged_codes, (unsigned long long)p.n_tiles,
             (unsigned long long)(n_rows - p.n_tiles * p.tile_rows));
  }
  return S2A_OK;
}

}  // extern "C"
