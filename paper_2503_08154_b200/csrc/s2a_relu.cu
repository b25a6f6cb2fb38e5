// ReLU with a 1-bit stash (Section 3.2, "ReLU layer"): the derivative is 0 or 1, so the
// backward pass needs one bit per element.  There are no rows and no reductions: a plain
// grid-stride kernel in which every thread owns one mask byte (8 consecutive elements) at
// a time, so that loads, stores and mask bytes of a warp are all contiguous.
#include "s2a_common.cuh"
#include "s2a_launch.h"

namespace s2a {
namespace {

constexpr int kThreads = 256;

// 8 consecutive elements of the I/O type.
template <int DT> struct Oct;
template <> struct Oct<kBF16> {
  uint4 r;
  __device__ __forceinline__ void load(const void* p, uint64_t b) { r = ((const uint4*)p)[b]; }
  __device__ __forceinline__ void store(void* p, uint64_t b) const { ((uint4*)p)[b] = r; }
  // keeps the elements whose mask bit is set, zeroes the others; returns the bits of (x > 0)
  __device__ __forceinline__ uint32_t positive_bits() const {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    uint32_t bits = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      // bfloat16 > 0: sign clear and magnitude non-zero
      const uint32_t lo = w[k] & 0xffffu, hi = w[k] >> 16;
      bits |= (uint32_t)(lo - 1u < 0x7fffu) << (2 * k);
      bits |= (uint32_t)(hi - 1u < 0x7fffu) << (2 * k + 1);
    }
    return bits;
  }
  __device__ __forceinline__ void keep(uint32_t bits) {
    uint32_t* w = &r.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t m = ((bits >> (2 * k)) & 1u ? 0x0000ffffu : 0u) | ((bits >> (2 * k + 1)) & 1u ? 0xffff0000u : 0u);
      w[k] &= m;
    }
  }
};
template <> struct Oct<kF32> {
  float4 a, b;
  __device__ __forceinline__ void load(const void* p, uint64_t i) { a = ((const float4*)p)[2 * i]; b = ((const float4*)p)[2 * i + 1]; }
  __device__ __forceinline__ void store(void* p, uint64_t i) const { ((float4*)p)[2 * i] = a; ((float4*)p)[2 * i + 1] = b; }
  __device__ __forceinline__ uint32_t positive_bits() const {
    return (a.x > 0.f) | (a.y > 0.f) << 1 | (a.z > 0.f) << 2 | (a.w > 0.f) << 3 | (b.x > 0.f) << 4 |
           (b.y > 0.f) << 5 | (b.z > 0.f) << 6 | (b.w > 0.f) << 7;
  }
  __device__ __forceinline__ void keep(uint32_t bits) {
    a.x = bits & 1u ? a.x : 0.f; a.y = bits & 2u ? a.y : 0.f; a.z = bits & 4u ? a.z : 0.f; a.w = bits & 8u ? a.w : 0.f;
    b.x = bits & 16u ? b.x : 0.f; b.y = bits & 32u ? b.y : 0.f; b.z = bits & 64u ? b.z : 0.f; b.w = bits & 128u ? b.w : 0.f;
  }
};

__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// FWD: in = x, out = y, mask written.  BWD: in = grad_out, out = grad_in, mask read.
template <int DT, bool FWD>
__global__ void __launch_bounds__(kThreads) relu_kernel(const void* in, void* out, uint8_t* mask, uint64_t n) {
  using T = typename Io<DT>::T;
  grid_launch_dependents();
  grid_dependency_wait();
  const uint64_t n8 = n >> 3;  // whole mask bytes
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  uint64_t b = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  // four independent bytes per round keep 64 (128) bytes of loads in flight per thread
  for (; b + 3 * stride < n8; b += 4 * stride) {
    Oct<DT> v[4];
    uint32_t bits[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k].load(in, b + k * stride);
    if (!FWD) {
#pragma unroll
      for (int k = 0; k < 4; ++k) bits[k] = mask[b + k * stride];
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (FWD) bits[k] = v[k].positive_bits();
      v[k].keep(bits[k]);
      v[k].store(out, b + k * stride);
      if (FWD) mask[b + k * stride] = (uint8_t)bits[k];
    }
  }
  for (; b < n8; b += stride) {
    Oct<DT> v;
    v.load(in, b);
    const uint32_t bits = FWD ? v.positive_bits() : mask[b];
    v.keep(bits);
    v.store(out, b);
    if (FWD) mask[b] = (uint8_t)bits;
  }
  // the last, partial byte
  if (blockIdx.x == 0 && threadIdx.x == 0 && (n & 7u)) {
    const T* x = (const T*)in;
    T* y = (T*)out;
    uint32_t bits = FWD ? 0u : mask[n8];
    for (uint64_t e = n8 << 3; e < n; ++e) {
      const float xe = Io<DT>::widen(x[e]);
      const uint32_t k = (uint32_t)(e & 7u);
      if (FWD) bits |= (uint32_t)(xe > 0.0f) << k;
      y[e] = Io<DT>::narrow((bits >> k) & 1u ? xe : 0.0f);
    }
    if (FWD) mask[n8] = (uint8_t)bits;
  }
}

int relu_grid(uint64_t n) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const uint64_t want = ((n >> 3) + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sms * 8;  // 8 resident CTAs of 256 threads per SM
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

template <int DT, bool FWD>
cudaError_t launch(const void* in, void* out, uint8_t* mask, uint64_t n, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(relu_grid(n));
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, relu_kernel<DT, FWD>, in, out, mask, n);
}

}  // namespace

cudaError_t launch_relu(bool fwd, int dt, const void* in, void* out, uint8_t* mask, uint64_t n, cudaStream_t st) {
  if (dt == kF32) return fwd ? launch<kF32, true>(in, out, mask, n, st) : launch<kF32, false>(in, out, mask, n, st);
  return fwd ? launch<kBF16, true>(in, out, mask, n, st) : launch<kBF16, false>(in, out, mask, n, st);
}

}  // namespace s2a
