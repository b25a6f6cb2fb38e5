// The activation-free pieces next to the stash path (Section 3.1): Channel Average Pooling
// forward/backward (Eq. 5) and the Low-Rank Prompt add (Eq. 3).  Plain memory-bound
// kernels: grid-stride, 16-byte accesses where the shape allows, scalar otherwise.
#include "s2a_common.cuh"
#include "s2a_launch.h"

namespace s2a {
namespace {

constexpr int kThreads = 256;

int grid_for(uint64_t work_items) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  uint64_t want = (work_items + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sms * 8;
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

__device__ __forceinline__ void widen8(const uint4& r, float* v) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    v[2 * k] = __uint_as_float(w[k] << 16);
    v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint4 narrow8(const float* v) {
  uint32_t w[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
    w[k] = *(uint32_t*)&b;
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// ---- CAP.  channels % r == 0, so groups of r consecutive elements never straddle a row and
// the tensor can be treated as flat: y[i] = mean(x[i r .. i r + r - 1]).  The sum runs in
// index order in binary32.  R8 = true is the paper's r = 8 with one (bfloat16) or two
// (binary32) 16-byte loads per output.
template <int DT, bool R8>
__global__ void __launch_bounds__(kThreads) cap_fwd_kernel(const void* xv, void* yv, uint64_t n_out, uint32_t r) {
  using T = typename Io<DT>::T;
  const T* x = (const T*)xv;
  T* y = (T*)yv;
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n_out; i += stride) {
    float sum = 0.0f;
    if (R8) {
      float v[8];
      if (DT == kBF16) {
        widen8(((const uint4*)xv)[i], v);
      } else {
        const float4 a = ((const float4*)xv)[2 * i], b = ((const float4*)xv)[2 * i + 1];
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) sum += v[j];
      y[i] = Io<DT>::narrow(sum * 0.125f);
    } else {
      for (uint32_t j = 0; j < r; ++j) sum += Io<DT>::widen(x[i * r + j]);
      y[i] = Io<DT>::narrow(__fdiv_rn(sum, (float)r));
    }
  }
}

template <int DT, bool R8>
__global__ void __launch_bounds__(kThreads) cap_bwd_kernel(const void* gv, void* ov, uint64_t n_out, uint32_t r) {
  using T = typename Io<DT>::T;
  const T* g = (const T*)gv;
  T* out = (T*)ov;
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  if (R8 && DT == kF32) {
    // one 16-byte store per thread, neighbours in a warp next to each other: thread q
    // writes one half of group q / 2
    for (uint64_t q = (uint64_t)blockIdx.x * kThreads + threadIdx.x; q < 2 * n_out; q += stride) {
      const float v = Io<DT>::widen(g[q >> 1]) * 0.125f;
      ((float4*)ov)[q] = make_float4(v, v, v, v);
    }
    return;
  }
  for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < n_out; i += stride) {
    const float gi = Io<DT>::widen(g[i]);
    if (R8) {
      const float v = gi * 0.125f;
      if (DT == kBF16) {
        float vv[8] = {v, v, v, v, v, v, v, v};
        ((uint4*)ov)[i] = narrow8(vv);
      } else {
        ((float4*)ov)[2 * i] = make_float4(v, v, v, v);
        ((float4*)ov)[2 * i + 1] = make_float4(v, v, v, v);
      }
    } else {
      const T v = Io<DT>::narrow(__fdiv_rn(gi, (float)r));
      for (uint32_t j = 0; j < r; ++j) out[i * r + j] = v;
    }
  }
}

// ---- LRP forward: y[b, t, c] = x[b, t, c] + sum_k A[t, k] B[k, c].  A thread owns the W
// consecutive channels of one token that fill 16 bytes: it forms its W prompt values once
// (binary32, k in order) and then streams over its share of the batch, four samples in
// flight at a time (y may alias x, but only element for element, so a thread's loads may
// run ahead of its own stores).  VEC = false is the scalar form for channel counts that are
// not a multiple of W.
template <int DT, bool VEC>
__global__ void __launch_bounds__(kThreads) lrp_fwd_kernel(const void* xv, const float* A, const float* B, void* yv,
                                                           uint32_t batch, uint32_t tokens, uint32_t channels,
                                                           uint32_t rank) {
  using T = typename Io<DT>::T;
  constexpr int W = VEC ? (DT == kBF16 ? 8 : 4) : 1;
  constexpr int kAhead = 4;
  const uint32_t cgroups = channels / W;
  const uint64_t items = (uint64_t)tokens * cgroups;
  const uint64_t item = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  if (item >= items) return;
  const uint32_t t = (uint32_t)(item / cgroups), c0 = (uint32_t)(item % cgroups) * W;
  float p[W];
#pragma unroll
  for (int w = 0; w < W; ++w) p[w] = 0.0f;
  for (uint32_t k = 0; k < rank; ++k) {
    const float a = A[(uint64_t)t * rank + k];
    if (VEC) {  // B is 16-byte aligned here and c0 a multiple of 4: whole float4 loads
      const float4* brow = (const float4*)(B + (uint64_t)k * channels + c0);
#pragma unroll
      for (int h = 0; h < W / 4; ++h) {
        const float4 bv = brow[h];
        p[4 * h] = fmaf(a, bv.x, p[4 * h]);
        p[(4 * h + 1) % W] = fmaf(a, bv.y, p[(4 * h + 1) % W]);
        p[(4 * h + 2) % W] = fmaf(a, bv.z, p[(4 * h + 2) % W]);
        p[(4 * h + 3) % W] = fmaf(a, bv.w, p[(4 * h + 3) % W]);
      }
    } else {
#pragma unroll
      for (int w = 0; w < W; ++w) p[w] = fmaf(a, B[(uint64_t)k * channels + c0 + w], p[w]);
    }
  }
  const uint64_t sample = (uint64_t)tokens * channels;
  const uint64_t e0 = (uint64_t)t * channels + c0;
  if (VEC) {
    const uint4* xin = (const uint4*)((const T*)xv + e0);
    uint4* yout = (uint4*)((T*)yv + e0);
    const uint64_t step = sample * sizeof(T) / 16;  // one sample, in 16-byte units
    for (uint32_t b = blockIdx.y; b < batch; b += gridDim.y * kAhead) {
      uint4 raw[kAhead];
#pragma unroll
      for (int j = 0; j < kAhead; ++j) {
        const uint32_t bj = b + j * gridDim.y;
        if (bj < batch) raw[j] = xin[bj * step];
      }
#pragma unroll
      for (int j = 0; j < kAhead; ++j) {
        const uint32_t bj = b + j * gridDim.y;
        if (bj >= batch) continue;
        if (DT == kBF16) {
          float v[8];
          widen8(raw[j], v);
#pragma unroll
          for (int w = 0; w < W; ++w) v[w] += p[w];
          yout[bj * step] = narrow8(v);
        } else {
          float4 v = *(float4*)&raw[j];
          v.x += p[0]; v.y += p[1 % W]; v.z += p[2 % W]; v.w += p[3 % W];
          yout[bj * step] = *(uint4*)&v;
        }
      }
    }
  } else {
    for (uint32_t b = blockIdx.y; b < batch; b += gridDim.y) {
      const uint64_t e = (uint64_t)b * sample + e0;
      ((T*)yv)[e] = Io<DT>::narrow(Io<DT>::widen(((const T*)xv)[e]) + p[0]);
    }
  }
}

// ---- LRP forward, tile form.  A CTA owns TILE consecutive elements of the flattened
// [tokens * channels] sample: every thread forms ONE prompt value (binary32, k in order) into
// shared memory -- once per CTA, whatever the batch -- then the CTA streams the batch through
// the tile, a thread keeping the prompt values of its own 16-byte chunk in registers and kAhead
// samples in flight.  The first samples are requested before the prompt is formed, so that their
// latency runs under that arithmetic.  Needs channels % W == 0 (whole 16-byte chunks per token).
constexpr int kLrpTile = 256;

template <int DT>
__global__ void __launch_bounds__(kThreads) lrp_tile_kernel(const void* xv, const float* A, const float* B, void* yv,
                                                            uint32_t batch, uint32_t channels, uint32_t rank,
                                                            uint64_t sample) {
  using T = typename Io<DT>::T;
  constexpr int W = DT == kBF16 ? 8 : 4;          // elements per 16 bytes
  constexpr int CH = kLrpTile / W;                // chunks per tile
  constexpr int SPR = kThreads / CH;              // samples a CTA touches per round
  constexpr int kAhead = 4;
  __shared__ __align__(16) float P[kLrpTile];
  const uint32_t chunk = threadIdx.x % CH, srow = threadIdx.x / CH;
  const uint64_t e0 = (uint64_t)blockIdx.x * kLrpTile + (uint64_t)chunk * W;   // this thread's chunk in the sample
  const bool mine = e0 < sample;
  const uint64_t step = sample * sizeof(T) / 16;  // one sample, in 16-byte units
  const uint4* xin = (const uint4*)((const T*)xv + e0);
  uint4* yout = (uint4*)((T*)yv + e0);
  const uint32_t b_first = blockIdx.y * SPR + srow, b_stride = gridDim.y * SPR;
  uint4 raw[kAhead];
#pragma unroll
  for (int j = 0; j < kAhead; ++j) {
    const uint32_t bj = b_first + j * b_stride;
    if (mine && bj < batch) raw[j] = xin[bj * step];
  }
  {
    const uint64_t e = (uint64_t)blockIdx.x * kLrpTile + threadIdx.x;
    float acc = 0.0f;
    if (e < sample) {
      const uint32_t t = (uint32_t)(e / channels), c = (uint32_t)(e % channels);
      const float* arow = A + (uint64_t)t * rank;
      const float* bcol = B + c;
#pragma unroll 6
      for (uint32_t k = 0; k < rank; ++k) acc = fmaf(arow[k], bcol[(uint64_t)k * channels], acc);
    }
    P[threadIdx.x] = acc;
  }
  __syncthreads();
  if (!mine) return;
  float p[W];
#pragma unroll
  for (int h = 0; h < W / 4; ++h) {
    const float4 v = ((const float4*)P)[chunk * (W / 4) + h];
    p[4 * h] = v.x; p[4 * h + 1] = v.y; p[4 * h + 2] = v.z; p[4 * h + 3] = v.w;
  }
  for (uint32_t b = b_first; b < batch; b += b_stride * kAhead) {
    if (b != b_first) {
#pragma unroll
      for (int j = 0; j < kAhead; ++j) {
        const uint32_t bj = b + j * b_stride;
        if (bj < batch) raw[j] = xin[bj * step];
      }
    }
#pragma unroll
    for (int j = 0; j < kAhead; ++j) {
      const uint32_t bj = b + j * b_stride;
      if (bj >= batch) continue;
      if (DT == kBF16) {
        float v[8];
        widen8(raw[j], v);
#pragma unroll
        for (int w = 0; w < W; ++w) v[w] += p[w];
        yout[bj * step] = narrow8(v);
      } else {
        float4 v = *(float4*)&raw[j];
        v.x += p[0]; v.y += p[1 % W]; v.z += p[2 % W]; v.w += p[3 % W];
        yout[bj * step] = *(uint4*)&v;
      }
    }
  }
}

}  // namespace

template <int DT>
void launch_cap_dt(bool fwd, bool r8, int grid, const void* in, void* out, uint64_t n_out, uint32_t r, cudaStream_t st) {
  if (fwd) {
    if (r8) cap_fwd_kernel<DT, true><<<grid, kThreads, 0, st>>>(in, out, n_out, r);
    else cap_fwd_kernel<DT, false><<<grid, kThreads, 0, st>>>(in, out, n_out, r);
  } else {
    if (r8) cap_bwd_kernel<DT, true><<<grid, kThreads, 0, st>>>(in, out, n_out, r);
    else cap_bwd_kernel<DT, false><<<grid, kThreads, 0, st>>>(in, out, n_out, r);
  }
}

cudaError_t launch_cap(bool fwd, int dt, const void* in, void* out, uint64_t n_out, uint32_t r, cudaStream_t st) {
  if (n_out == 0) return cudaSuccess;
  const int grid = grid_for(n_out);
  if (dt == kF32) launch_cap_dt<kF32>(fwd, r == 8, grid, in, out, n_out, r, st);
  else launch_cap_dt<kBF16>(fwd, r == 8, grid, in, out, n_out, r, st);
  return cudaGetLastError();
}

cudaError_t launch_lrp_fwd(int dt, const void* x, const float* A, const float* B, void* y, uint32_t batch,
                           uint32_t tokens, uint32_t channels, uint32_t rank, cudaStream_t st) {
  if ((uint64_t)batch * tokens * channels == 0) return cudaSuccess;
  const uint32_t w = dt == kF32 ? 4u : 8u;  // channels in 16 bytes
  if (channels % w == 0 && dt == kBF16) {
    // tile form (bfloat16; measured slower than the per-thread form below in binary32: 4.7 against
    // 5.1 TB/s on [256, 197, 768]): the prompt is formed once per CTA; the batch is split over gridDim.y only as
    // far as it takes to give every SM four CTAs, and never below kAhead rounds per thread
    const uint64_t sample = (uint64_t)tokens * channels;
    const uint64_t tiles = (sample + kLrpTile - 1) / kLrpTile;
    const uint32_t spr = kThreads / (kLrpTile / w);
    uint64_t splits = (148ull * 4 + tiles - 1) / tiles;
    const uint64_t most = batch / (spr * 4) > 0 ? batch / (spr * 4) : 1;
    if (splits > most) splits = most;
    if (splits > 65535) splits = 65535;
    if (tiles <= 0x7fffffffull) {
      dim3 grid((unsigned)tiles, (unsigned)splits);
      lrp_tile_kernel<kBF16><<<grid, kThreads, 0, st>>>(x, A, B, y, batch, channels, rank, sample);
      return cudaGetLastError();
    }
  }
  const bool vec = channels % w == 0 && ((uintptr_t)B & 15u) == 0;  // the vector form reads B 16 bytes at a time
  const uint64_t items = (uint64_t)tokens * (vec ? channels / w : channels);
  // The batch is split over gridDim.y.  Each split forms its prompt values again (rank
  // multiply-adds per element of one sample), so only as many splits as give every SM a
  // thousand threads: with four samples in flight per thread that covers the memory latency.
  uint64_t splits = (148ull * 1024 + items - 1) / items;
  if (splits > batch) splits = batch;
  if (splits > 64) splits = 64;
  if (splits < 1) splits = 1;
  dim3 grid((unsigned)((items + kThreads - 1) / kThreads), (unsigned)splits);
  if (dt == kF32) {
    if (vec) lrp_fwd_kernel<kF32, true><<<grid, kThreads, 0, st>>>(x, A, B, y, batch, tokens, channels, rank);
    else lrp_fwd_kernel<kF32, false><<<grid, kThreads, 0, st>>>(x, A, B, y, batch, tokens, channels, rank);
  } else {
    if (vec) lrp_fwd_kernel<kBF16, true><<<grid, kThreads, 0, st>>>(x, A, B, y, batch, tokens, channels, rank);
    else lrp_fwd_kernel<kBF16, false><<<grid, kThreads, 0, st>>>(x, A, B, y, batch, tokens, channels, rank);
  }
  return cudaGetLastError();
}

}  // namespace s2a
