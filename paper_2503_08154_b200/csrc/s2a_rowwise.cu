// Row-at-a-time kernels: one CTA walks one row (two rows when row_len is odd, so that
// the CTA owns whole code bytes) straight from global memory, with scalar accesses and
// several passes over the row.  They accept any row length and any row alignment and
// serve (a) the ragged rows left over after the pipelined tiles and (b) shapes whose
// rows do not fit a shared-memory tile.  Correctness first; the pipelined kernels in
// s2a_tile.cu carry the bandwidth.
#include "s2a_common.cuh"
#include "s2a_launch.h"

namespace s2a {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct BlockScratch {
  float red[2][kWarps];
  float bcast[2];
};

// OP: 0 max, 1 min, 2 sum.  All threads get the result.
template <int OP>
__device__ __forceinline__ float block_reduce(float v, BlockScratch& sc, int slot) {
  if (OP == 0) v = warp_max(v);
  if (OP == 1) v = warp_min(v);
  if (OP == 2) v = warp_sum(v);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) sc.red[slot][w] = v;
  __syncthreads();
  if (w == 0) {
    float t = l < kWarps ? sc.red[slot][l] : (OP == 0 ? -INFINITY : (OP == 1 ? INFINITY : 0.0f));
    if (OP == 0) t = warp_max(t);
    if (OP == 1) t = warp_min(t);
    if (OP == 2) t = warp_sum(t);
    if (l == 0) sc.bcast[slot] = t;
  }
  __syncthreads();
  float r = sc.bcast[slot];
  __syncthreads();
  return r;
}

__device__ __forceinline__ uint32_t nibble_at(const uint8_t* codes, uint64_t e) {
  uint32_t b = codes[e >> 1];
  return (e & 1) ? (b >> 4) : (b & 0xFu);
}

template <int KERNEL, int DT>
__global__ void __launch_bounds__(kThreads) rowwise_kernel(RowwiseArgs a) {
  using T = typename Io<DT>::T;
  constexpr int ACT = act_of(KERNEL);
  constexpr float kActClip = Act<ACT>::kClipOf;
  __shared__ BlockScratch sc;
  __shared__ float row_mn[2], row_inv[2], row_s[2], row_aux[2];
  __shared__ float dtab[2][16];

  const T* in = (const T*)a.in;
  T* out = (T*)a.out;
  const uint32_t L = a.row_len;
  const uint32_t P = (L & 1u) ? 2u : 1u;
  const uint64_t n_groups = (a.n_rows + P - 1) / P;
  const int tid = threadIdx.x;

  for (uint64_t g = blockIdx.x; g < n_groups; g += gridDim.x) {
    const uint64_t r0 = a.row0 + g * P;
    const uint64_t rows_left = a.row0 + a.n_rows - r0;
    const uint32_t rows_here = rows_left < P ? (uint32_t)rows_left : P;
    const uint64_t e0 = r0 * L;  // even by construction
    const uint64_t cnt = (uint64_t)rows_here * L;

    // ---- per-row statistics ---------------------------------------------------
    for (uint32_t h = 0; h < rows_here; ++h) {
      const uint64_t base = e0 + (uint64_t)h * L;
      if (is_act_fwd(KERNEL)) {
        float mn = INFINITY, mx = -INFINITY;
        for (uint32_t i = tid; i < L; i += kThreads) {
          float x = Io<DT>::widen(in[base + i]);
          mn = fminf(mn, x);
          mx = fmaxf(mx, x);
        }
        mn = block_reduce<1>(mn, sc, 0);
        mx = block_reduce<0>(mx, sc, 1);
        // min/max of the clipped row = clipped min/max of the row (the clip is monotone)
        QRange q = make_qrange(fminf(fmaxf(mn, -kActClip), kActClip), fminf(fmaxf(mx, -kActClip), kActClip));
        if (tid == 0) { row_mn[h] = q.mn; row_inv[h] = q.inv; row_s[h] = q.s; }
      } else if (KERNEL == kSoftmaxFwd) {
        float m = -INFINITY;
        for (uint32_t i = tid; i < L; i += kThreads) m = fmaxf(m, Io<DT>::widen(in[base + i]));
        m = block_reduce<0>(m, sc, 0);
        float z = 0.0f;
        for (uint32_t i = tid; i < L; i += kThreads) z += expf(Io<DT>::widen(in[base + i]) - m);
        z = block_reduce<2>(z, sc, 1);
        const float rz = __fdiv_rn(1.0f, z);
        float mn = INFINITY, mx = -INFINITY;
        for (uint32_t i = tid; i < L; i += kThreads) {
          float y = expf(Io<DT>::widen(in[base + i]) - m) * rz;
          T yo = Io<DT>::narrow(y);
          out[base + i] = yo;           // same index as the read: in-place is safe
          float v = Io<DT>::widen(yo);  // the value as written is what gets quantised
          mn = fminf(mn, v);
          mx = fmaxf(mx, v);
        }
        mn = block_reduce<1>(mn, sc, 0);
        mx = block_reduce<0>(mx, sc, 1);
        QRange q = make_qrange(mn, mx);
        if (tid == 0) { row_mn[h] = q.mn; row_inv[h] = q.inv; row_s[h] = q.s; }
      } else if (is_act_bwd(KERNEL)) {
        const float mn = a.meta[2 * (r0 + h)], s = a.meta[2 * (r0 + h) + 1];
        if (tid < 16) dtab[h][tid] = (float)act_derivative<ACT>((uint32_t)tid, mn, s);
      } else {  // kSoftmaxBwd
        const float mn = a.meta[2 * (r0 + h)], s = a.meta[2 * (r0 + h) + 1];
        float dot = 0.0f;
        for (uint32_t i = tid; i < L; i += kThreads) {
          float yh = dequant(nibble_at(a.codes, base + i), mn, s);
          dot = fmaf(Io<DT>::widen(in[base + i]), yh, dot);
        }
        dot = block_reduce<2>(dot, sc, 0);
        if (tid == 0) { row_mn[h] = mn; row_s[h] = s; row_aux[h] = dot; }
      }
    }
    __syncthreads();  // statistics in shared memory, and forward outputs, now visible

    if (is_fwd(KERNEL) && tid < (int)rows_here) {
      a.meta[2 * (r0 + tid)] = row_mn[tid];
      a.meta[2 * (r0 + tid) + 1] = row_s[tid];
    }

    // ---- element pass, one code byte (two flat-adjacent elements) per step --------
    const uint64_t n_bytes = (cnt + 1) >> 1;
    for (uint64_t b = tid; b < n_bytes; b += kThreads) {
      uint32_t byte = 0;
      if (!is_fwd(KERNEL)) byte = a.codes[(e0 >> 1) + b];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const uint64_t rel = 2 * b + k;
        if (rel < cnt) {
          const uint32_t h = rel >= L ? 1u : 0u;
          const uint64_t e = e0 + rel;
          if (is_act_fwd(KERNEL)) {
            float x = Io<DT>::widen(in[e]);
            QRange q{row_mn[h], row_inv[h], row_s[h]};
            byte |= quant_code(fminf(fmaxf(x, -kActClip), kActClip), q) << (4 * k);
            out[e] = Io<DT>::narrow(act_value<ACT>(x));
          } else if (KERNEL == kSoftmaxFwd) {
            QRange q{row_mn[h], row_inv[h], row_s[h]};
            byte |= quant_code(Io<DT>::widen(out[e]), q) << (4 * k);
          } else if (is_act_bwd(KERNEL)) {
            uint32_t code = (byte >> (4 * k)) & 0xFu;
            out[e] = Io<DT>::narrow(Io<DT>::widen(in[e]) * dtab[h][code]);
          } else {
            uint32_t code = (byte >> (4 * k)) & 0xFu;
            float yh = dequant(code, row_mn[h], row_s[h]);
            out[e] = Io<DT>::narrow(yh * (Io<DT>::widen(in[e]) - row_aux[h]));
          }
        }
      }
      if (is_fwd(KERNEL)) a.codes[(e0 >> 1) + b] = (uint8_t)byte;
    }
    __syncthreads();  // shared statistics are reused by the next group
  }
}

template <int KERNEL, int DT>
cudaError_t launch_one(const RowwiseArgs& a, cudaStream_t st) {
  const uint32_t P = (a.row_len & 1u) ? 2u : 1u;
  uint64_t groups = (a.n_rows + P - 1) / P;
  unsigned grid = (unsigned)(groups < (1ull << 20) ? groups : (1ull << 20));
  rowwise_kernel<KERNEL, DT><<<grid, kThreads, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rowwise(int kernel, int dt, const RowwiseArgs& a, cudaStream_t st) {
  if (a.n_rows == 0) return cudaSuccess;
#define S2A_CASE(K) \
  case K:           \
    return dt == kF32 ? launch_one<K, kF32>(a, st) : launch_one<K, kBF16>(a, st);
  switch (kernel) {
    S2A_CASE(kGeluFwd)
    S2A_CASE(kGeluBwd)
    S2A_CASE(kSoftmaxFwd)
    S2A_CASE(kSoftmaxBwd)
    S2A_CASE(kSiluFwd)
    S2A_CASE(kSiluBwd)
  }
#undef S2A_CASE
  return cudaErrorInvalidValue;
}

}  // namespace s2a
