// Row-at-a-time kernels: one team of threads walks one row (or the few rows that end on a
// whole code byte when row_len is odd, so that the team owns whole code bytes) straight from global memory, with scalar accesses and
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

// A team is the whole CTA (long rows) or one warp (short rows, eight teams per CTA).
struct TeamScratch {
  float red[2][kWarps];
  float bcast[2];
};

template <int TEAM>
__device__ __forceinline__ void team_sync() {
  if (TEAM == 32) __syncwarp();
  else __syncthreads();
}

// OP: 0 max, 1 min, 2 sum.  All threads of the team get the result.
template <int OP, int TEAM>
__device__ __forceinline__ float team_reduce(float v, TeamScratch& sc, int slot) {
  if (OP == 0) v = warp_max(v);
  if (OP == 1) v = warp_min(v);
  if (OP == 2) v = warp_sum(v);
  if (TEAM == 32) return v;
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

// The N-bit code of flat element e: bits [(e N) mod 8, +N) of byte (e N) / 8.
template <int NBITS>
__device__ __forceinline__ uint32_t code_at(const uint8_t* codes, uint64_t e) {
  constexpr uint32_t EPB = 8 / NBITS;
  const uint32_t b = codes[e / EPB];
  return (b >> ((uint32_t)(e % EPB) * NBITS)) & ((1u << NBITS) - 1u);
}

// NBITS is the code width of Eq. 8 (4 in the paper; 2 and 8 are the general-N form).
// A team owns the smallest group of rows that ends on a whole code byte: 8 / NBITS elements
// share a byte, so up to 4 rows when NBITS = 2 and row_len is odd.
template <int KERNEL, int DT, int NBITS, int TEAM>
__global__ void __launch_bounds__(kThreads) rowwise_kernel(RowwiseArgs a) {
  using T = typename Io<DT>::T;
  constexpr int ACT = act_of(KERNEL);
  constexpr float kActClip = Act<ACT>::kClipOf;
  constexpr uint32_t EPB = 8 / NBITS;                 // elements per code byte
  constexpr uint32_t kMask = (1u << NBITS) - 1u;
  constexpr float kLevelsN = (float)((1 << NBITS) - 1);
  constexpr int kTab = 1 << NBITS;
  constexpr int kTeams = kThreads / TEAM;
  __shared__ TeamScratch sc;  // used by whole-CTA teams only
  __shared__ float s_mn[kTeams][4], s_inv[kTeams][4], s_s[kTeams][4], s_aux[kTeams][4];
  __shared__ float s_dtab[kTeams][is_act_bwd(KERNEL) ? 4 : 1][is_act_bwd(KERNEL) ? kTab : 1];
  const int team = threadIdx.x / TEAM;
  float* row_mn = s_mn[team];
  float* row_inv = s_inv[team];
  float* row_s = s_s[team];
  float* row_aux = s_aux[team];
  float (*dtab)[is_act_bwd(KERNEL) ? kTab : 1] = s_dtab[team];

  const T* in = (const T*)a.in;
  T* out = (T*)a.out;
  const uint32_t L = a.row_len;
  uint32_t P = 1;                                     // rows per group: P * L is a multiple of EPB
  while ((P * (uint64_t)L) % EPB != 0) P *= 2;
  const uint64_t n_groups = (a.n_rows + P - 1) / P;
  const int tid = threadIdx.x % TEAM;
  // Launched with programmatic stream serialization: let the next kernel of the stream set
  // up while this one runs, and touch no global memory before the previous one has finished.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  for (uint64_t g = (uint64_t)blockIdx.x * kTeams + team; g < n_groups; g += (uint64_t)gridDim.x * kTeams) {
    const uint64_t r0 = a.row0 + g * P;
    const uint64_t rows_left = a.row0 + a.n_rows - r0;
    const uint32_t rows_here = rows_left < P ? (uint32_t)rows_left : P;
    const uint64_t e0 = r0 * L;  // a multiple of EPB by construction
    const uint64_t cnt = (uint64_t)rows_here * L;

    // ---- per-row statistics ---------------------------------------------------
    for (uint32_t h = 0; h < rows_here; ++h) {
      const uint64_t base = e0 + (uint64_t)h * L;
      if (is_act_fwd(KERNEL)) {
        float mn = INFINITY, mx = -INFINITY;
        for (uint32_t i = tid; i < L; i += TEAM) {
          float x = Io<DT>::widen(in[base + i]);
          mn = fminf(mn, x);
          mx = fmaxf(mx, x);
        }
        mn = team_reduce<1, TEAM>(mn, sc, 0);
        mx = team_reduce<0, TEAM>(mx, sc, 1);
        // min/max of the clipped row = clipped min/max of the row (the clip is monotone)
        QRange q = make_qrange(fminf(fmaxf(mn, -kActClip), kActClip), fminf(fmaxf(mx, -kActClip), kActClip), kLevelsN);
        if (tid == 0) { row_mn[h] = q.mn; row_inv[h] = q.inv; row_s[h] = q.s; }
      } else if (KERNEL == kSoftmaxFwd) {
        float m = -INFINITY;
        for (uint32_t i = tid; i < L; i += TEAM) m = fmaxf(m, Io<DT>::widen(in[base + i]));
        m = team_reduce<0, TEAM>(m, sc, 0);
        float z = 0.0f;
        for (uint32_t i = tid; i < L; i += TEAM) z += expf(Io<DT>::widen(in[base + i]) - m);
        z = team_reduce<2, TEAM>(z, sc, 1);
        const float rz = __fdiv_rn(1.0f, z);
        float mn = INFINITY, mx = -INFINITY;
        for (uint32_t i = tid; i < L; i += TEAM) {
          float y = expf(Io<DT>::widen(in[base + i]) - m) * rz;
          T yo = Io<DT>::narrow(y);
          out[base + i] = yo;           // same index as the read: in-place is safe
          float v = Io<DT>::widen(yo);  // the value as written is what gets quantised
          mn = fminf(mn, v);
          mx = fmaxf(mx, v);
        }
        mn = team_reduce<1, TEAM>(mn, sc, 0);
        mx = team_reduce<0, TEAM>(mx, sc, 1);
        QRange q = make_qrange(mn, mx, kLevelsN);
        if (tid == 0) { row_mn[h] = q.mn; row_inv[h] = q.inv; row_s[h] = q.s; }
      } else if (is_act_bwd(KERNEL)) {
        const float mn = a.meta[2 * (r0 + h)], s = a.meta[2 * (r0 + h) + 1];
        for (int c = tid; c < kTab; c += TEAM) dtab[h][c] = (float)act_derivative<ACT>((uint32_t)c, mn, s);
      } else {  // kSoftmaxBwd
        const float mn = a.meta[2 * (r0 + h)], s = a.meta[2 * (r0 + h) + 1];
        float dot = 0.0f;
        for (uint32_t i = tid; i < L; i += TEAM) {
          float yh = dequant(code_at<NBITS>(a.codes, base + i), mn, s);
          dot = fmaf(Io<DT>::widen(in[base + i]), yh, dot);
        }
        dot = team_reduce<2, TEAM>(dot, sc, 0);
        if (tid == 0) { row_mn[h] = mn; row_s[h] = s; row_aux[h] = dot; }
      }
    }
    team_sync<TEAM>();  // statistics in shared memory, and forward outputs, now visible

    if (is_fwd(KERNEL) && tid < (int)rows_here) {
      a.meta[2 * (r0 + tid)] = row_mn[tid];
      a.meta[2 * (r0 + tid) + 1] = row_s[tid];
    }

    // ---- element pass, one code byte (EPB flat-adjacent elements) per step ----------
    const uint64_t n_bytes = (cnt + EPB - 1) / EPB;
    for (uint64_t b = tid; b < n_bytes; b += TEAM) {
      uint32_t byte = 0;
      if (!is_fwd(KERNEL)) byte = a.codes[e0 / EPB + b];
#pragma unroll
      for (uint32_t k = 0; k < EPB; ++k) {
        const uint64_t rel = EPB * b + k;
        if (rel < cnt) {
          const uint32_t h = (uint32_t)(rel / L);
          const uint64_t e = e0 + rel;
          if (is_act_fwd(KERNEL)) {
            float x = Io<DT>::widen(in[e]);
            QRange q{row_mn[h], row_inv[h], row_s[h]};
            byte |= quant_code(fminf(fmaxf(x, -kActClip), kActClip), q, kMask) << (NBITS * k);
            out[e] = Io<DT>::narrow(act_value<ACT>(x));
          } else if (KERNEL == kSoftmaxFwd) {
            QRange q{row_mn[h], row_inv[h], row_s[h]};
            byte |= quant_code(Io<DT>::widen(out[e]), q, kMask) << (NBITS * k);
          } else if (is_act_bwd(KERNEL)) {
            uint32_t code = (byte >> (NBITS * k)) & kMask;
            out[e] = Io<DT>::narrow(Io<DT>::widen(in[e]) * dtab[h][code]);
          } else {
            uint32_t code = (byte >> (NBITS * k)) & kMask;
            float yh = dequant(code, row_mn[h], row_s[h]);
            out[e] = Io<DT>::narrow(yh * (Io<DT>::widen(in[e]) - row_aux[h]));
          }
        }
      }
      if (is_fwd(KERNEL)) a.codes[e0 / EPB + b] = (uint8_t)byte;
    }
    team_sync<TEAM>();  // shared statistics are reused by the next group
  }
}

template <int KERNEL, int DT, int NBITS>
cudaError_t launch_one(const RowwiseArgs& a, cudaStream_t st) {
  uint32_t P = 1;
  while ((P * (uint64_t)a.row_len) % (8 / NBITS) != 0) P *= 2;
  const uint64_t groups = (a.n_rows + P - 1) / P;
  // a warp per group while a lane's share stays small, else the whole CTA per group
  const bool warp_teams = (uint64_t)P * a.row_len <= 2048;
  const uint64_t ctas = warp_teams ? (groups + kWarps - 1) / kWarps : groups;
  const unsigned grid = (unsigned)(ctas < (1ull << 20) ? ctas : (1ull << 20));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (warp_teams) return cudaLaunchKernelEx(&cfg, rowwise_kernel<KERNEL, DT, NBITS, 32>, a);
  return cudaLaunchKernelEx(&cfg, rowwise_kernel<KERNEL, DT, NBITS, kThreads>, a);
}

template <int KERNEL, int DT>
cudaError_t launch_bits(int bits, const RowwiseArgs& a, cudaStream_t st) {
  if (bits == 4) return launch_one<KERNEL, DT, 4>(a, st);
  if (KERNEL <= kSoftmaxBwd) {  // the general-N form exists for the four kernels of the paper
    constexpr int K = KERNEL <= kSoftmaxBwd ? KERNEL : kGeluFwd;
    if (bits == 2) return launch_one<K, DT, 2>(a, st);
    if (bits == 8) return launch_one<K, DT, 8>(a, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_rowwise(int kernel, int dt, const RowwiseArgs& a, cudaStream_t st, int bits) {
  if (a.n_rows == 0) return cudaSuccess;
#define S2A_CASE(K) \
  case K:           \
    return dt == kF32 ? launch_bits<K, kF32>(bits, a, st) : launch_bits<K, kBF16>(bits, a, st);
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
