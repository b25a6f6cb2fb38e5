// GELU forward whose 4-bit stash uses ONE quantiser range for the whole tensor (the other
// reading of Section 3.2, "GeLU layer": the paragraph quantises the clipped input over its
// min-to-max range and leaves open over which elements that range is taken).
// The range must be known before the first code can be formed, so the tensor is read twice:
//   1. range_partials: one CTA per chunk of 65,536 elements writes the chunk's (min, max)
//      of x into scratch memory;
//   2. range_final: one CTA folds the partials into scratch[0..1];
//   3. fixed_range_fwd: an elementwise pass writes y, the codes and every row's (min, s).
// Scratch layout (floats): [0] min, [1] max, then one (min, max) pair per chunk.
// Algorithmic bytes: 2 reads of x + y + codes (6.5 B per bfloat16 element, 12.5 B per
// binary32 element) against 4.5 / 8.5 for the per-row stash.
#include "s2a_common.cuh"
#include "s2a_launch.h"

#include <atomic>

namespace s2a {
namespace {

constexpr int kThreads = 256;
constexpr uint32_t kChunk = 65536;  // elements per partial; a multiple of 8 * kThreads

struct Red {
  float red[2][kThreads / 32];
};

__device__ __forceinline__ void block_minmax(float& mn, float& mx, Red& sc) {
  mn = warp_min(mn);
  mx = warp_max(mx);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sc.red[0][w] = mn; sc.red[1][w] = mx; }
  __syncthreads();
  if (w == 0) {
    mn = l < kThreads / 32 ? sc.red[0][l] : INFINITY;
    mx = l < kThreads / 32 ? sc.red[1][l] : -INFINITY;
    mn = warp_min(mn);
    mx = warp_max(mx);
  }
}

template <int DT>
__device__ __forceinline__ void load8(const void* p, uint64_t oct, float* v) {
  if (DT == kBF16) {
    const uint4 r = ((const uint4*)p)[oct];
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v[2 * k] = __uint_as_float(w[k] << 16);
      v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  } else {
    const float4 a = ((const float4*)p)[2 * oct], b = ((const float4*)p)[2 * oct + 1];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <int DT>
__device__ __forceinline__ void store8(void* p, uint64_t oct, const float* v) {
  if (DT == kBF16) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
      w[k] = *(uint32_t*)&b;
    }
    ((uint4*)p)[oct] = make_uint4(w[0], w[1], w[2], w[3]);
  } else {
    ((float4*)p)[2 * oct] = make_float4(v[0], v[1], v[2], v[3]);
    ((float4*)p)[2 * oct + 1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads) range_partials(const void* x, uint64_t n, float* scratch) {
  using T = typename Io<DT>::T;
  __shared__ Red sc;
  const uint64_t e0 = (uint64_t)blockIdx.x * kChunk;
  const uint64_t e1 = e0 + kChunk < n ? e0 + kChunk : n;
  float mn = INFINITY, mx = -INFINITY;
  const uint64_t oct0 = e0 >> 3, oct1 = e1 >> 3;  // whole groups of 8 (e0 is a multiple of 8)
  for (uint64_t o = oct0 + threadIdx.x; o < oct1; o += kThreads) {
    float v[8];
    load8<DT>(x, o, v);
#pragma unroll
    for (int k = 0; k < 8; ++k) { mn = fminf(mn, v[k]); mx = fmaxf(mx, v[k]); }
  }
  for (uint64_t e = (oct1 << 3) + threadIdx.x; e < e1; e += kThreads) {
    const float v = Io<DT>::widen(((const T*)x)[e]);
    mn = fminf(mn, v);
    mx = fmaxf(mx, v);
  }
  block_minmax(mn, mx, sc);
  if (threadIdx.x == 0) { scratch[2 + 2 * blockIdx.x] = mn; scratch[3 + 2 * blockIdx.x] = mx; }
}

__global__ void __launch_bounds__(kThreads) range_final(float* scratch, uint32_t n_chunks) {
  __shared__ Red sc;
  float mn = INFINITY, mx = -INFINITY;
  for (uint32_t c = threadIdx.x; c < n_chunks; c += kThreads) {
    mn = fminf(mn, scratch[2 + 2 * c]);
    mx = fmaxf(mx, scratch[3 + 2 * c]);
  }
  block_minmax(mn, mx, sc);
  // min / max of the clipped tensor = clipped min / max of the tensor (the clip is monotone)
  if (threadIdx.x == 0) {
    scratch[0] = fminf(fmaxf(mn, -kClip), kClip);
    scratch[1] = fminf(fmaxf(mx, -kClip), kClip);
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads) fixed_range_fwd(const void* x, void* y, uint8_t* codes, float* meta,
                                                            const float* scratch, uint64_t n, uint64_t n_rows) {
  using T = typename Io<DT>::T;
  const QRange q = make_qrange(scratch[0], scratch[1]);
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  const uint64_t tid = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  for (uint64_t r = tid; r < n_rows; r += stride) {
    meta[2 * r] = q.mn;
    meta[2 * r + 1] = q.s;
  }
  const uint64_t n8 = n >> 3;
  for (uint64_t o = tid; o < n8; o += stride) {
    float v[8];
    load8<DT>(x, o, v);
    uint32_t bits = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      bits |= quant_code(fminf(fmaxf(v[k], -kClip), kClip), q) << (4 * k);
      v[k] = gelu_eval<DT>(v[k]);
    }
    store8<DT>(y, o, v);
    ((uint32_t*)codes)[o] = bits;
  }
  if (tid == 0 && (n & 7u)) {  // the ragged end: fewer than 8 elements
    uint32_t bits = 0;
    for (uint64_t e = n8 << 3; e < n; ++e) {
      const float xe = Io<DT>::widen(((const T*)x)[e]);
      bits |= quant_code(fminf(fmaxf(xe, -kClip), kClip), q) << (4 * (e & 7u));
      ((T*)y)[e] = Io<DT>::narrow(gelu_eval<DT>(xe));
    }
    for (uint64_t b = n8 * 4; b < (n + 1) / 2; ++b) codes[b] = (uint8_t)(bits >> (8 * (b - n8 * 4)));
  }
}

// Scratch of the allocation-free entry point: room for the range partials of
// kStaticChunks chunks.  It lives in every GPU that loads the library, from load to exit,
// and is shared by all calls of that entry point on the device.
constexpr uint32_t kStaticChunks = 8192;  // 8192 * 65,536 = 536,870,912 elements at most
static __device__ __align__(256) float g_static_range_scratch[2 + 2 * kStaticChunks];  // 65,544 bytes

}  // namespace

uint64_t tensor_range_static_max_elems() { return (uint64_t)kStaticChunks * kChunk; }

// In host code `g_static_range_scratch` is only a handle for the runtime, not an address
// the GPU understands: the device address is looked up once per device (with that device
// current) and that pointer is what the kernels receive.
cudaError_t launch_gelu_fwd_tensor_range_static(int dt, const void* x, void* y, uint8_t* codes, float* meta,
                                                uint64_t n, uint64_t n_rows, cudaStream_t st) {
  static std::atomic<float*> device_address[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  float* scratch = device_address[dev].load(std::memory_order_acquire);
  if (scratch == nullptr) {
    // two threads making the first call on a device both look the address up and store the
    // same value; the address stays valid until the device is reset
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_range_scratch);
    if (e != cudaSuccess) return e;
    scratch = (float*)p;
    device_address[dev].store(scratch, std::memory_order_release);
  }
  // Nothing in the scratch has to start at zero: the first kernel overwrites the partial of
  // every chunk this call uses, the second overwrites the folded range, the third only reads.
  return launch_gelu_fwd_tensor_range(dt, x, y, codes, meta, scratch, n, n_rows, st);
}

uint64_t tensor_range_scratch_bytes(uint64_t n) {
  return 8 + 8 * ((n + kChunk - 1) / kChunk);
}

cudaError_t launch_gelu_fwd_tensor_range(int dt, const void* x, void* y, uint8_t* codes, float* meta, float* scratch,
                                         uint64_t n, uint64_t n_rows, cudaStream_t st) {
  const uint32_t n_chunks = (uint32_t)((n + kChunk - 1) / kChunk);
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  uint64_t want = ((n >> 3) + kThreads - 1) / kThreads;
  if (want < 1) want = 1;
  const unsigned grid = (unsigned)(want < (uint64_t)sms * 8 ? want : (uint64_t)sms * 8);
  if (dt == kF32) {
    range_partials<kF32><<<n_chunks, kThreads, 0, st>>>(x, n, scratch);
    range_final<<<1, kThreads, 0, st>>>(scratch, n_chunks);
    fixed_range_fwd<kF32><<<grid, kThreads, 0, st>>>(x, y, codes, meta, scratch, n, n_rows);
  } else {
    range_partials<kBF16><<<n_chunks, kThreads, 0, st>>>(x, n, scratch);
    range_final<<<1, kThreads, 0, st>>>(scratch, n_chunks);
    fixed_range_fwd<kBF16><<<grid, kThreads, 0, st>>>(x, y, codes, meta, scratch, n, n_rows);
  }
  return cudaGetLastError();
}

}  // namespace s2a
